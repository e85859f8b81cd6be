"""GPU parity of the index-set union (Sec. 3.6 Eq. 7; Alg. 1 Phase 3) against the CPU oracle: integer work, so the
positions and the set sizes must agree exactly."""
import numpy as np
import pytest
import torch

import oracle as O
import paper_2601_17702_b200 as S

pytestmark = pytest.mark.gpu


def _dev():
    assert torch.cuda.is_available()
    return torch.device("cuda:0")


def gpu_fuse(centers, w, lexical, lead, tail, L, cap):
    d = _dev()
    c = torch.from_numpy(np.ascontiguousarray(centers, dtype=np.int32)).to(d)
    lx = None if lexical is None else torch.from_numpy(np.ascontiguousarray(lexical, dtype=np.int32)).to(d)
    ws = torch.zeros(S.s3_fuse_workspace_bytes(c.shape[0], L), dtype=torch.uint8, device=d)
    idx, cnt = S.s3_fuse_index_sets(c, w, lx, lead, tail, L, cap, ws)
    torch.cuda.synchronize()
    return idx.cpu().numpy(), cnt.cpu().numpy()


def check(centers, w, lexical, lead, tail, L, cap):
    idx, cnt = gpu_fuse(centers, w, lexical, lead, tail, L, cap)
    want = O.fuse_index_sets(centers, w, lexical, lead, tail, L)
    for q, m in enumerate(want):
        assert cnt[q] == len(m), (q, cnt[q], len(m))
        n = min(cap, len(m))
        np.testing.assert_array_equal(idx[q, :n], m[:n])
        assert (idx[q, n:] == -1).all()


def test_hand_example():
    # window 6 around centres 10 and 13 = 7..15, lexical {3, 14, 39}, lead 2, tail 3 of L = 40 (worked by hand)
    idx, cnt = gpu_fuse(np.array([[10, 13, -1]]), 6, np.array([[3, 14, 39, 50, -1]]), 2, 3, 40, 32)
    assert cnt[0] == 15
    assert idx[0, :15].tolist() == [0, 1, 3, 7, 8, 9, 10, 11, 12, 13, 14, 15, 37, 38, 39]
    assert (idx[0, 15:] == -1).all()


@pytest.mark.parametrize("L,Q,N,w,n_lex,lead,tail", [
    (1000, 3, 8, 64, 20, 16, 16),          # several words, ragged tail word
    (131072, 4, 32, 256, 128, 64, 64),     # the 128K context of the retrieval workload
    (70001, 2, 100, 33, 0, 0, 0),          # odd width, no lexical set, no lead/tail
    (513, 2, 4, 2000, 7, 600, 600),        # windows and lead/tail wider than the context
    (31, 1, 3, 4, 5, 1, 1),                # a single partial word
])
def test_parity(L, Q, N, w, n_lex, lead, tail):
    rng = np.random.default_rng(L + N)
    centers = rng.integers(-1, L, size=(Q, N))
    centers[:, ::5] = np.minimum(centers[:, ::5], 3)          # some windows clipped at position 0
    centers[:, 1::7] = L - 1                                   # and at the end
    lexical = rng.integers(-2, L + 10, size=(Q, n_lex)) if n_lex else None
    check(centers, w, lexical, lead, tail, L, cap=L)


def test_cap_truncates_and_counts():
    rng = np.random.default_rng(5)
    centers = rng.integers(0, 5000, size=(2, 16))
    check(centers, 128, None, 8, 8, 5000, cap=100)
    check(centers, 128, None, 8, 8, 5000, cap=0)


def test_degenerate_sets():
    check(np.full((2, 4), -1), 64, None, 0, 0, 4096, cap=16)          # nothing selected: empty sets
    check(np.zeros((3, 0), dtype=np.int32), 64, None, 4, 4, 4096, cap=16)  # no centre columns, bias only
    check(np.array([[5]]), 0, np.array([[7, 7, 7]]), 0, 0, 64, cap=8)  # zero-width windows, repeated lexical hits
    check(np.array([[5]]), 3, None, 2, 2, 0, cap=8)                    # empty context


def test_error_paths():
    d = _dev()
    c = torch.zeros((1, 2), dtype=torch.int32, device=d)
    ws = torch.zeros(S.s3_fuse_workspace_bytes(1, 4096) - 1, dtype=torch.uint8, device=d)
    with pytest.raises(S.S3Error):
        S.s3_fuse_index_sets(c, 8, None, 0, 0, 4096, 16, ws)
    ws = torch.zeros(S.s3_fuse_workspace_bytes(1, 4096), dtype=torch.uint8, device=d)
    with pytest.raises(S.S3Error):
        S.s3_fuse_index_sets(c, -1, None, 0, 0, 4096, 16, ws)
    with pytest.raises(S.S3Error):
        S.s3_fuse_index_sets(c, 8, None, 0, 0, 1 << 40, 16, ws)
