"""Failure paths that need no GPU fault: a status word planted from the host is mapped to the error the kernels'
bounded waits and input checks would report, and a pinned-memory reservation that cannot succeed fails with an
error code and leaves the index usable. Nothing here makes a kernel's wait run out or touches invalid memory."""
import ctypes as C

import numpy as np
import pytest
import torch

import oracle as O
import paper_2601_17702_b200 as S
from paper_2601_17702_b200 import binding as B
from parity import csr_equal

pytestmark = pytest.mark.gpu


def _dev():
    assert torch.cuda.is_available()
    return torch.device("cuda:0")


@pytest.mark.parametrize("code,status", [
    (1, B.S3_ERR_TIMEOUT),        # MMA warp: operand tile never arrived
    (2, B.S3_ERR_TIMEOUT),        # TMA warp: pipeline slot never freed
    (3, B.S3_ERR_TIMEOUT),        # epilogue: accumulator never completed
    (4, B.S3_ERR_TIMEOUT),        # MMA warp: accumulator never drained
    (16, B.S3_ERR_INVALID_ARG),   # postings: feature id >= d_sae
    (17, B.S3_ERR_CAPACITY),      # compact index: buffer too small
    (18, B.S3_ERR_INVALID_ARG),   # postings: repeated id in a token
])
def test_planted_status_word_maps_to_its_error(code, status):
    d = _dev()
    ws = S.new_workspace(256, d)
    raw = C.c_uint32(123)
    stream = C.c_void_p(torch.cuda.current_stream().cuda_stream)
    assert B.lib().s3_workspace_status(C.c_void_p(ws.data_ptr()), stream, C.byref(raw)) == B.S3_OK and raw.value == 0
    ws[:4] = torch.tensor(list(int(code).to_bytes(4, "little")), dtype=torch.uint8, device=d)      # host -> device copy
    assert B.lib().s3_workspace_status(C.c_void_p(ws.data_ptr()), stream, C.byref(raw)) == status
    assert raw.value == code
    assert str(code) in B.s3_last_error()
    with pytest.raises(B.S3Error) as e:
        S.s3_workspace_status(ws)
    assert e.value.code == status
    # the word is sticky until the caller clears it; afterwards the workspace reads clean again
    ws[:4] = 0
    assert S.s3_workspace_status(ws) == 0


def test_impossible_pinned_reservation_fails_and_the_index_stays_usable():
    d = _dev()
    d_sae, T, k = 64, 100, 4
    ix = S.Index(1, d_sae, 1 << 16)
    with pytest.raises(B.S3Error) as e:
        ix.reserve(1 << 60)                      # no machine has an exbibyte of pinned memory: the allocator refuses
    assert e.value.code in (B.S3_ERR_NOMEM, B.S3_ERR_CUDA)
    assert "pinned reservation" in str(e.value)
    rng = np.random.default_rng(1)
    ids = np.stack([rng.choice(d_sae, size=k, replace=False) for _ in range(T)]).astype(np.int32)
    row_ptr = torch.zeros(d_sae + 1, dtype=torch.int32, device=d)
    pos = torch.zeros(T * k, dtype=torch.int32, device=d)
    ws = S.new_workspace(S.s3_postings_workspace_bytes(T, k, d_sae), d)
    S.s3_postings_build(torch.as_tensor(ids).to(d), d_sae, 0, row_ptr, pos, ws)
    ix.append(0, row_ptr, pos, T, k, 0)          # a normal append after the failed reservation
    rp, ps, _ = ix.export_csr(0)
    orp, opos, _ = O.postings(ids, d_sae, 0)
    csr_equal(rp.numpy(), ps.numpy(), orp, opos)
    assert ix.stats()["n_postings"] == T * k
    with pytest.raises(B.S3Error) as e:          # and the ordering check still works
        ix.append(0, row_ptr, pos, T, k, 10)
    assert e.value.code == B.S3_ERR_STATE
    ix.close()
