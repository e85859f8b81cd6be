"""CPU oracle of the streaming-scan hot path. TEST INFRASTRUCTURE ONLY.

Only tests/, the smoke check and the benchmark's CPU-baseline leg may import this package; the
product package never does. The floating-point arithmetic lives in s3_oracle.cpp (plain C++, fp64), which this file
marshals numpy arrays into; the pure integer / set steps at the end of the file (index-set union, compact index
encoding) are plain Python here. No function is "parity unpinned".
"""
from __future__ import annotations

import ctypes as C

import numpy as np

from .build import build as _build

_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(_build())
        _lib.s3o_idf.restype = C.c_double
        _lib.s3o_idf.argtypes = [C.c_double]
        _lib.s3o_num_threads.restype = C.c_int
    return _lib


def _p(a, t):
    return None if a is None else a.ctypes.data_as(C.POINTER(t))


def _f32(a):
    return np.ascontiguousarray(np.asarray(a, dtype=np.float32))


def _i32(a):
    return np.ascontiguousarray(np.asarray(a, dtype=np.int32))


def num_threads() -> int:
    return int(lib().s3o_num_threads())


def preact(x, W, b_enc, b_dec) -> np.ndarray:
    """Eq. 1 before the ReLU, fp64 [T, d_sae]."""
    x, W, b_enc, b_dec = _f32(x), _f32(W), _f32(b_enc), _f32(b_dec)
    T, d_in = x.shape
    d_sae = W.shape[1]
    assert W.shape[0] == d_in and b_enc.shape == (d_sae,) and b_dec.shape == (d_in,)
    pre = np.empty((T, d_sae), dtype=np.float64)
    lib().s3o_preact(_p(x, C.c_float), _p(W, C.c_float), _p(b_enc, C.c_float), _p(b_dec, C.c_float),
                     C.c_int64(T), C.c_int(d_in), C.c_int(d_sae), _p(pre, C.c_double))
    return pre


def topk(pre, k: int):
    """ReLU + Top-k (Eq. 1-3): ids int32 [T,k] (pad -1), vals fp32 [T,k] (pad 0)."""
    pre = np.ascontiguousarray(pre, dtype=np.float64)
    T, d_sae = pre.shape
    ids = np.empty((T, k), dtype=np.int32)
    vals = np.empty((T, k), dtype=np.float32)
    lib().s3o_topk(_p(pre, C.c_double), C.c_int64(T), C.c_int(d_sae), C.c_int(k), _p(ids, C.c_int32), _p(vals, C.c_float))
    return ids, vals


def encode_topk(x, W, b_enc, b_dec, k: int):
    return topk(preact(x, W, b_enc, b_dec), k)


def decode(ids, vals, W_dec, b_dec, x=None):
    """x_hat = z_hat W_dec + b_dec (Sec. 3.3, after Eq. 2), fp64 [T, d_in]; with x also the per-token squared
    reconstruction error, fp64 [T]. ids int32 [T,k] (-1 = padding), vals fp32 [T,k], W_dec [d_sae, d_in]."""
    ids, vals, W_dec, b_dec = _i32(ids), _f32(vals), _f32(W_dec), _f32(b_dec)
    T, k = ids.shape
    d_sae, d_in = W_dec.shape
    assert vals.shape == ids.shape and b_dec.shape == (d_in,) and ids.max(initial=-1) < d_sae
    x_hat = np.empty((T, d_in), dtype=np.float64)
    xx = None if x is None else _f32(x)
    err = None if x is None else np.empty(T, dtype=np.float64)
    lib().s3o_decode(_p(ids, C.c_int32), _p(vals, C.c_float), C.c_int64(T), C.c_int(k), _p(W_dec, C.c_float),
                     _p(b_dec, C.c_float), C.c_int(d_in), C.c_int(d_sae), _p(xx, C.c_float), _p(x_hat, C.c_double),
                     _p(err, C.c_double))
    return x_hat if x is None else (x_hat, err)


def postings(ids, d_sae: int, pos_base: int = 0, vals=None):
    """Eq. 4 for one chunk: (row_ptr uint32 [d_sae+1], pos int32 [nnz], pval fp32 [nnz] or None)."""
    ids = _i32(ids)
    T, k = ids.shape
    v = None if vals is None else _f32(vals)
    row_ptr = np.empty(d_sae + 1, dtype=np.uint32)
    pos = np.empty(max(T * k, 1), dtype=np.int32)
    pval = None if v is None else np.empty(max(T * k, 1), dtype=np.float32)
    lib().s3o_postings(_p(ids, C.c_int32), _p(v, C.c_float), C.c_int64(T), C.c_int(k), C.c_int(d_sae),
                       C.c_int64(pos_base), _p(row_ptr, C.c_uint32), _p(pos, C.c_int32), _p(pval, C.c_float))
    nnz = int(row_ptr[-1])
    return row_ptr, pos[:nnz].copy(), (None if pval is None else pval[:nnz].copy())


def index_merge(chunks, d_sae: int):
    """Concatenate per-chunk CSRs [(row_ptr, pos), ...] (arrival order) into one CSR per layer."""
    n = len(chunks)
    rps = [np.ascontiguousarray(c[0], dtype=np.uint32) for c in chunks]
    pss = [np.ascontiguousarray(c[1], dtype=np.int32) for c in chunks]
    total = int(sum(int(r[-1]) for r in rps))
    row_ptr = np.empty(d_sae + 1, dtype=np.uint64)
    pos = np.empty(max(total, 1), dtype=np.int32)
    RP = (C.POINTER(C.c_uint32) * n)(*[_p(r, C.c_uint32) for r in rps])
    PP = (C.POINTER(C.c_int32) * n)(*[_p(p if p.size else np.zeros(1, np.int32), C.c_int32) for p in pss])
    lib().s3o_index_merge(C.c_int(n), RP, PP, C.c_int(d_sae), _p(row_ptr, C.c_uint64), _p(pos, C.c_int32))
    return row_ptr, pos[:total].copy()


def idf(freq: float) -> float:
    return float(lib().s3o_idf(C.c_double(freq)))


def score_spans(ctx_ids, q_ids, q_vals, d_sae: int, width: int, stride: int, mode: int = 0, stop_freq: int = 0):
    """ctx_ids [n_layers, L, k]; q_ids/q_vals [n_layers, Q, nq, kq]. Returns int64 coact [Q,n_spans]
    (mode 0) or fp64 weighted scores (mode 1)."""
    ctx_ids, q_ids, q_vals = _i32(ctx_ids), _i32(q_ids), _f32(q_vals)
    n_layers, L, k = ctx_ids.shape
    _, Q, nq, kq = q_ids.shape
    assert q_ids.shape[0] == n_layers and q_vals.shape == q_ids.shape
    ns = (L - width) // stride + 1 if L >= width else 0
    co = np.zeros((Q, ns), dtype=np.int64) if mode == 0 else None
    ws = np.zeros((Q, ns), dtype=np.float64) if mode == 1 else None
    lib().s3o_score_spans(_p(ctx_ids, C.c_int32), C.c_int64(L), C.c_int(k), C.c_int(d_sae), C.c_int(n_layers),
                          _p(q_ids, C.c_int32), _p(q_vals, C.c_float), C.c_int(Q), C.c_int(nq), C.c_int(kq),
                          C.c_int(width), C.c_int(stride), C.c_int(mode), C.c_int64(stop_freq),
                          _p(co, C.c_int64), _p(ws, C.c_double))
    return co if mode == 0 else ws


def fuse_select(base, bm25, alpha: float, beta: float, s: int):
    """base: int64 coact or fp64 weighted scores [Q, n_spans]; bm25 fp32 [Q, n_spans] or None.
    Returns (top_idx int32 [Q,s], top_score fp32 [Q,s], all_scores fp32 [Q,n_spans])."""
    base = np.ascontiguousarray(base)
    Q, ns = base.shape
    co = base if base.dtype == np.int64 else None
    ws = base.astype(np.float64) if co is None else None
    b = None if bm25 is None else _f32(bm25)
    top_idx = np.empty((Q, s), dtype=np.int32)
    top_score = np.empty((Q, s), dtype=np.float32)
    allsc = np.empty((Q, max(ns, 1)), dtype=np.float32)
    lib().s3o_fuse_select(_p(co, C.c_int64), _p(ws, C.c_double), _p(b, C.c_float), C.c_float(alpha), C.c_float(beta),
                          C.c_int(Q), C.c_int64(ns), C.c_int(s), _p(top_idx, C.c_int32), _p(top_score, C.c_float),
                          _p(allsc, C.c_float))
    return top_idx, top_score, allsc[:, :ns]


def position_density(ctx_ids, q_ids, q_vals, d_sae: int, conv_kernel: int, nms_radius: int, n_centers: int,
                     stop_freq: int = 0):
    """Per-position relevance S (Eq. 6), its box-smoothed density S' and the NMS peak positions.
    ctx_ids [n_layers, L, k]; q_ids/q_vals [n_layers, Q, nq, kq].
    Returns (S fp64 [Q,L], D fp64 [Q,L], centers int32 [Q,n_centers] (-1 = none), center_density fp32 [Q,n_centers])."""
    ctx_ids, q_ids, q_vals = _i32(ctx_ids), _i32(q_ids), _f32(q_vals)
    n_layers, L, k = ctx_ids.shape
    _, Q, nq, kq = q_ids.shape
    assert q_ids.shape[0] == n_layers and q_vals.shape == q_ids.shape
    S = np.zeros((Q, L), dtype=np.float64)
    D = np.zeros((Q, L), dtype=np.float64)
    centers = np.empty((Q, n_centers), dtype=np.int32)
    dens = np.empty((Q, n_centers), dtype=np.float32)
    lib().s3o_position_density(_p(ctx_ids, C.c_int32), C.c_int64(L), C.c_int(k), C.c_int(d_sae), C.c_int(n_layers),
                               _p(q_ids, C.c_int32), _p(q_vals, C.c_float), C.c_int(Q), C.c_int(nq), C.c_int(kq),
                               C.c_int(conv_kernel), C.c_int(nms_radius), C.c_int(n_centers), C.c_int64(stop_freq),
                               _p(S, C.c_double), _p(D, C.c_double), _p(centers, C.c_int32), _p(dens, C.c_float))
    return S, D, centers, dens


def fuse_index_sets(centers, span_width: int, lexical, lead: int, tail: int, L: int):
    """Sec. 3.6, Eq. 7: M_final = M_S3 U M_BM25 U M_Bias, per query, as ascending unique positions in [0, L).
    M_S3   = union over the selected centres c >= 0 of the window [c - span_width//2, c - span_width//2 + span_width)
             (reading: the paper's variable-length span rule is not given; a fixed window centred on the peak stands in),
    M_BM25 = the supplied lexical positions (entries < 0 are padding; entries >= L are ignored),
    M_Bias = the first `lead` and the last `tail` positions.
    centers [Q, N] int, lexical [Q, n_lex] int or None. Returns a list of Q int32 arrays. Plain Python sets."""
    centers = np.asarray(centers)
    out = []
    for q in range(centers.shape[0]):
        m = set()
        for c in centers[q].tolist():
            if c >= 0:
                lo = c - span_width // 2
                m.update(t for t in range(lo, lo + span_width) if 0 <= t < L)
        if lexical is not None:
            m.update(int(t) for t in np.asarray(lexical)[q].tolist() if 0 <= t < L)
        m.update(range(0, min(lead, L)))
        m.update(range(max(0, L - tail), L))
        out.append(np.array(sorted(m), dtype=np.int32))
    return out


# ---------------------------------------------------------------------------------------------- compact index
# Sec. 3.4 (memory analysis) asks a production index for contiguous integer arrays with delta encoding and optional
# stop-feature pruning; the layout itself is this library's (the paper fixes none). Per layer, from the merged CSR:
#   pruning   : a feature whose list is longer than stop_freq > 0 keeps no postings;
#   row_ptr   : uint64 [D+1], prefix sum of the kept list lengths;
#   blocks    : a kept list is cut into blocks of 32 postings (the last one shorter); blk_ptr uint32 [D+1] is the prefix
#               sum of the lists' block counts;
#   per block : blk_first = its first position; width = bit length of the largest (gap - 1) between consecutive
#               positions inside the block (0 when all gaps are 1 or the block holds one posting);
#               blk_desc = (word offset of its payload << 6) | width;
#   payload   : uint32 words; a block of c postings stores its c - 1 values (gap - 1), `width` bits each, back to
#               back starting at bit 0 of its first word, least significant bit first, in ceil((c-1)*width/32)
#               words; blocks follow each other in order; one zero word closes the array.

def compact_encode(row_ptr, pos, stop_freq: int = 0):
    """Returns dict(row_ptr uint64 [D+1], blk_ptr uint32 [D+1], blk_first int32 [B], blk_desc uint64 [B],
    payload uint32 [W+1]). Python integers as bit buffers: slow and plain."""
    row_ptr = np.asarray(row_ptr, dtype=np.uint64)
    pos = np.asarray(pos, dtype=np.int64)
    D = len(row_ptr) - 1
    out_rp, blk_ptr, firsts, descs, words = [0], [0], [], [], []
    for f in range(D):
        lst = pos[int(row_ptr[f]):int(row_ptr[f + 1])].tolist()
        if stop_freq > 0 and len(lst) > stop_freq:
            lst = []
        out_rp.append(out_rp[-1] + len(lst))
        blk_ptr.append(blk_ptr[-1] + (len(lst) + 31) // 32)
        for b0 in range(0, len(lst), 32):
            blk = lst[b0:b0 + 32]
            gaps = [blk[i] - blk[i - 1] - 1 for i in range(1, len(blk))]
            assert all(g >= 0 for g in gaps), "positions of a list must ascend strictly"
            width = max(gaps).bit_length() if gaps else 0
            bits = 0
            for i, g in enumerate(gaps):
                bits |= g << (i * width)
            n_words = (len(gaps) * width + 31) // 32
            firsts.append(blk[0])
            descs.append((len(words) << 6) | width)
            words.extend((bits >> (32 * w)) & 0xFFFFFFFF for w in range(n_words))
    words.append(0)
    return dict(row_ptr=np.array(out_rp, dtype=np.uint64), blk_ptr=np.array(blk_ptr, dtype=np.uint32),
                blk_first=np.array(firsts, dtype=np.int32), blk_desc=np.array(descs, dtype=np.uint64),
                payload=np.array(words, dtype=np.uint32))


def compact_decode(c):
    """Inverse of compact_encode on the kept postings: (row_ptr uint64 [D+1], pos int32). Reads the payload bit by
    bit (written without reference to the encoder's buffer arithmetic)."""
    rp, bp = c["row_ptr"], c["blk_ptr"]
    payload = c["payload"]
    pos = []
    for f in range(len(rp) - 1):
        n = int(rp[f + 1]) - int(rp[f])
        for j, b in enumerate(range(int(bp[f]), int(bp[f + 1]))):
            cnt = min(32, n - 32 * j)
            desc = int(c["blk_desc"][b])
            width, bit = desc & 63, (desc >> 6) * 32
            p = int(c["blk_first"][b])
            pos.append(p)
            for _ in range(cnt - 1):
                g = 0
                for i in range(width):
                    g |= ((int(payload[(bit + i) // 32]) >> ((bit + i) % 32)) & 1) << i
                bit += width
                p += g + 1
                pos.append(p)
    return np.asarray(rp, dtype=np.uint64), np.array(pos, dtype=np.int32)


def prune_stop_features(row_ptr, pos, stop_freq: int):
    """The CSR with every list longer than stop_freq > 0 emptied (Sec. 3.4 stop-feature pruning; the appendix's
    hard frequency threshold applied when the index is built)."""
    row_ptr = np.asarray(row_ptr, dtype=np.uint64)
    pos = np.asarray(pos)
    keep, out_rp = [], [0]
    for f in range(len(row_ptr) - 1):
        lo, hi = int(row_ptr[f]), int(row_ptr[f + 1])
        if stop_freq > 0 and hi - lo > stop_freq:
            hi = lo
        keep.append(pos[lo:hi])
        out_rp.append(out_rp[-1] + hi - lo)
    return np.array(out_rp, dtype=np.uint64), (np.concatenate(keep) if keep else pos[:0]).astype(np.int32)


# ---------------------------------------------------------------------------------------------- head aggregation
def head_aggregate(ids, vals, k_out: int):
    """Sec. 3.3 / 3.4: the SAE reads one head's projection (x in R^d_head), while Sec. 3.4 counts k features per token
    once the heads have been aggregated; the aggregation rule is not given. Reading: all heads share one feature-ID space;
    a token's activation of feature f is the sum over the heads whose Top-k holds f (fp32, heads in ascending order,
    which is the precision the selection is made in), and the token keeps the k_out largest sums > 0, ordered by
    (sum descending, id ascending), padded with id -1 / value 0.
    ids int32 [T, H, k] (-1 = padding), vals fp32 [T, H, k]. Returns (ids int32 [T, k_out], vals fp32 [T, k_out])."""
    ids, vals = _i32(ids), _f32(vals)
    T, H, k = ids.shape
    out_i = np.full((T, k_out), -1, dtype=np.int32)
    out_v = np.zeros((T, k_out), dtype=np.float32)
    for t in range(T):
        acc = {}
        for h in range(H):
            for j in range(k):
                f = int(ids[t, h, j])
                if f >= 0:
                    acc[f] = np.float32(acc.get(f, np.float32(0.0)) + vals[t, h, j])
        best = sorted(((f, v) for f, v in acc.items() if v > 0), key=lambda fv: (-float(fv[1]), fv[0]))[:k_out]
        for r, (f, v) in enumerate(best):
            out_i[t, r], out_v[t, r] = f, v
    return out_i, out_v


# ---------------------------------------------------------------------------------------------- SAE training step
# The paper trains its Top-K SAEs with Adam (appendix table: learning rate 1e-3, batches of 4096 tokens) and gives no loss;
# reading: the mean over the batch of the squared reconstruction error of Sec. 3.3's x_hat, differentiated through the
# Top-k code with the active set held fixed (the selection is piecewise constant, so this is the gradient wherever it
# exists). Adam as published (Kingma & Ba): m = b1 m + (1-b1) g, v = b2 v + (1-b2) g^2, p -= lr * m_hat / (sqrt(v_hat) + eps)
# with m_hat = m / (1 - b1^step), v_hat = v / (1 - b2^step). Plain numpy, fp64.

def sae_loss_and_grads(x, W_enc, b_enc, W_dec, b_dec, ids):
    """x [T, d_in], W_enc [d_in, d_sae], b_enc [d_sae], W_dec [d_sae, d_in], b_dec [d_in], ids int32 [T, k] (the active
    set, -1 = padding). z[t,j] = W_enc[:, f]·(x_t - b_dec) + b_enc[f] for f = ids[t,j] (the pre-activation of a selected
    feature, which the ReLU passes), x_hat = z W_dec + b_dec, loss = mean_t ||x_hat_t - x_t||^2.
    Returns (loss, gW_enc, gb_enc, gW_dec, gb_dec), all fp64."""
    x = np.asarray(x, np.float64)
    W_enc, b_enc = np.asarray(W_enc, np.float64), np.asarray(b_enc, np.float64)
    W_dec, b_dec = np.asarray(W_dec, np.float64), np.asarray(b_dec, np.float64)
    ids = np.asarray(ids)
    T, d_in = x.shape
    gW_enc, gb_enc = np.zeros_like(W_enc), np.zeros_like(b_enc)
    gW_dec, gb_dec = np.zeros_like(W_dec), np.zeros_like(b_dec)
    loss = 0.0
    for t in range(T):
        f = ids[t][ids[t] >= 0]
        xc = x[t] - b_dec
        z = xc @ W_enc[:, f] + b_enc[f]
        r = z @ W_dec[f] + b_dec - x[t]
        loss += float(r @ r) / T
        g = 2.0 * r / T                                  # d loss / d x_hat_t
        gz = W_dec[f] @ g                                # d loss / d z
        np.add.at(gW_dec, f, np.outer(z, g))
        np.add.at(gb_enc, f, gz)
        np.add.at(gW_enc.T, f, np.outer(gz, xc))
        gb_dec += g - W_enc[:, f] @ gz                   # directly, and through (x - b_dec) in the encoder
    return loss, gW_enc, gb_enc, gW_dec, gb_dec


def adam_update(p, m, v, g, lr, beta1, beta2, eps, step):
    """One Adam update (step counted from 1). Returns (p, m, v), fp64."""
    p, m, v, g = (np.asarray(a, np.float64) for a in (p, m, v, g))
    m = beta1 * m + (1.0 - beta1) * g
    v = beta2 * v + (1.0 - beta2) * g * g
    m_hat = m / (1.0 - beta1 ** step)
    v_hat = v / (1.0 - beta2 ** step)
    return p - lr * m_hat / (np.sqrt(v_hat) + eps), m, v
