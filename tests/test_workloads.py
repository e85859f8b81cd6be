"""The seeded generators: reproducible, sliceable, and shaped like the stated distributions."""
import numpy as np
import torch

import oracle as O
from workloads import configs as C, generators as G


def test_rows_regenerate_independently():
    inp = C.ScanInputs(C.CFG2)
    a = inp.x("key", 0, 0, 300)
    b = inp.x("key", 0, 100, 50)
    assert torch.equal(a[100:150], b)
    assert not torch.equal(inp.x("key", 1, 0, 8), a[:8])      # layers are separate streams


def test_normal_moments_and_table():
    g = G.normal(1, G.TID_X, 0, 4000, 64).double()
    assert abs(g.mean()) < 0.01 and abs(g.std() - 1.0) < 0.01
    assert abs((g ** 4).mean() - 3.0) < 0.1


def test_unit_norm_columns_and_biases():
    w, b_enc, b_dec = G.sae_weights(0, 0, 128, 1024, torch.float32)
    assert torch.allclose((w.double() ** 2).sum(0), torch.ones(1024, dtype=torch.float64), atol=1e-5)
    assert abs(b_enc.std() - 0.1) < 0.01 and abs(b_dec.std() - 0.05) < 0.02


def test_channel_scale_outliers():
    s = G.channel_scale(2, 1024, 0.5, 0.01, 8.0)
    base = G.channel_scale(2, 1024, 0.5, 0.0, 1.0)
    ratio = (s / base)
    assert int((ratio > 7.9).sum()) == 11 and int((ratio < 1.1).sum()) == 1024 - 11
    assert abs(torch.log(base).std() - 0.5) < 0.05


def test_gamma21_moments():
    b = G.gamma21(4, 64, 512).double()
    assert abs(b.mean() - 2.0) < 0.05 and abs(b.var() - 2.0) < 0.15 and b.min() > 0


def test_zipf_ranks_follow_power_law():
    r = G.zipf_ranks(5, 0, 0, 200000, 64, 1.1)
    cnt = torch.bincount(r, minlength=64).double()
    slope = np.polyfit(np.log(np.arange(1, 33)), np.log(cnt[:32].numpy()), 1)[0]
    assert abs(slope + 1.1) < 0.1


def test_cfg1_oracle_scan_invariants():
    cfg = C.CFG1
    inp = C.ScanInputs(cfg)
    w, b_enc, b_dec = inp.sae("key", 0)
    x = inp.x("key", 0, 0, cfg.L)
    ids, vals = O.encode_topk(x.numpy(), w.numpy(), b_enc.numpy(), b_dec.numpy(), cfg.key.k)
    assert (ids >= 0).all()                       # every token has k positive activations here
    row_ptr, pos, _ = O.postings(ids, cfg.key.d_sae, 0)
    assert int(row_ptr[-1]) == cfg.L * cfg.key.k  # P = L * layers * k with one layer
    for f in (0, 17, 1023):
        lst = pos[row_ptr[f]:row_ptr[f + 1]]
        assert (np.diff(lst) > 0).all()


def test_cfg5_popular_features_are_popular():
    cfg = C.CFG5
    inp = C.ScanInputs(cfg)
    w, b_enc, b_dec = inp.sae("key", 0)
    x = inp.x("key", 0, 0, 1024)
    ids, _ = O.encode_topk(x.float().numpy(), w.float().numpy(), b_enc.numpy(), b_dec.numpy(), cfg.key.k)
    pi = G.zipf_popular_features(cfg.seed, 0, cfg.key.d_sae, cfg.zipf_ranks)
    cnt = np.bincount(ids[ids >= 0], minlength=cfg.key.d_sae)
    top = int(pi[0])
    assert cnt[top] > 20 * cnt.mean() and cnt[top] >= cnt[int(pi[8])]
