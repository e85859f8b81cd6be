"""The five seeded synthetic workloads (shapes only; values come from workloads.generators).

They stand in for the paper's long-context settings (LongBench-length contexts and the
128k-token stress test on Llama-3.1-8B, with 4 instrumented layers and chunked streaming):
same tensor shapes, sparsity k and chunking, synthetic values.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import torch

from . import generators as G


@dataclass(frozen=True)
class SaeShape:
    d_in: int
    d_sae: int
    k: int


@dataclass(frozen=True)
class ScanConfig:
    name: str
    seed: int
    L: int                 # context tokens
    chunk: int             # tokens per streamed chunk
    n_layers: int
    key: SaeShape
    query: SaeShape | None = None     # a second, throughput-only SAE over query projections
    dtype: torch.dtype = torch.bfloat16
    scale_sigma: float = 0.0          # lognormal per-channel scale
    outlier_frac: float = 0.0
    outlier_gain: float = 1.0
    zipf_ranks: int = 0               # > 0: Zipf-skewed low-rank mean shift
    zipf_exponent: float = 1.1
    zipf_gain: float = 4.0

    @property
    def n_chunks(self) -> int:
        return (self.L + self.chunk - 1) // self.chunk


@dataclass(frozen=True)
class RetrievalConfig:
    name: str
    scan: ScanConfig       # the index being searched
    Q: int                 # batched queries
    nq: int                # query tokens per query
    kq: int                # Top-k used for the query tokens
    width: int
    stride: int
    s: int                 # spans returned
    alpha: float
    beta: float            # 0 => no lexical fusion
    bm25_seed: int = 0


CFG1 = ScanConfig("cfg1_tiny", seed=0, L=2048, chunk=2048, n_layers=1,
                  key=SaeShape(128, 1024, 8), dtype=torch.float32)
CFG2 = ScanConfig("cfg2_llama8b_32k", seed=2, L=32768, chunk=4096, n_layers=1,
                  key=SaeShape(1024, 16384, 32), scale_sigma=0.5, outlier_frac=0.01, outlier_gain=8.0)
CFG3 = ScanConfig("cfg3_128k_4layers_kq", seed=3, L=131072, chunk=8192, n_layers=4,
                  key=SaeShape(1024, 16384, 32), query=SaeShape(4096, 32768, 64))
CFG5 = ScanConfig("cfg5_1m_qwen7b_zipf", seed=5, L=1048576, chunk=16384, n_layers=8,
                  key=SaeShape(512, 8192, 16), zipf_ranks=64)

CFG1_RETR = RetrievalConfig("cfg1_retrieval", CFG1, Q=1, nq=16, kq=8, width=64, stride=64, s=4,
                            alpha=1.0, beta=0.0)
CFG4 = RetrievalConfig("cfg4_retrieval_s16", CFG2, Q=256, nq=64, kq=64, width=64, stride=16, s=16,
                       alpha=0.5, beta=0.5, bm25_seed=4)
CFG4_S64 = RetrievalConfig("cfg4_retrieval_s64", CFG2, Q=256, nq=64, kq=64, width=64, stride=64, s=16,
                           alpha=0.5, beta=0.5, bm25_seed=4)

SCAN_CONFIGS = {c.name: c for c in (CFG1, CFG2, CFG3, CFG5)}
RETRIEVAL_CONFIGS = {c.name: c for c in (CFG1_RETR, CFG4, CFG4_S64)}


def n_spans(L: int, width: int, stride: int) -> int:
    return (L - width) // stride + 1 if L >= width else 0


class ScanInputs:
    """Lazily generated tensors of one scan workload (weights cached per layer and SAE)."""

    def __init__(self, cfg: ScanConfig, device="cpu"):
        self.cfg = cfg
        self.device = device
        self._sae: dict[tuple[str, int], tuple] = {}
        self._scale = None
        if cfg.scale_sigma > 0 or cfg.outlier_frac > 0:
            self._scale = G.channel_scale(cfg.seed, cfg.key.d_in, cfg.scale_sigma,
                                          cfg.outlier_frac, cfg.outlier_gain)

    def sae(self, which: str, layer: int):
        """(W_enc [d_in, d_sae], b_enc [d_sae] fp32, b_dec [d_in] fp32) of the key or query SAE."""
        key = (which, layer)
        if key not in self._sae:
            shp = self.cfg.key if which == "key" else self.cfg.query
            seed = self.cfg.seed + (0 if which == "key" else 500009)
            self._sae[key] = G.sae_weights(seed, layer, shp.d_in, shp.d_sae, self.cfg.dtype, self.device)
        return self._sae[key]

    def x(self, which: str, layer: int, row0: int, n_rows: int, device=None) -> torch.Tensor:
        """Rows row0 .. row0+n_rows-1 of the layer's key (or query) projection matrix."""
        cfg = self.cfg
        device = self.device if device is None else device
        if which == "key":
            if cfg.zipf_ranks:
                w = self.sae("key", layer)[0]
                return G.zipf_shifted_activations(cfg.seed, layer, row0, n_rows, w, cfg.zipf_ranks,
                                                  cfg.zipf_exponent, cfg.zipf_gain, cfg.dtype, device)
            return G.activations(cfg.seed, layer, row0, n_rows, cfg.key.d_in, cfg.dtype, self._scale, device)
        return G.activations(cfg.seed + 500009, layer, row0, n_rows, cfg.query.d_in, cfg.dtype, None,
                             device, tid=G.TID_QUERY_X)

    def retrieval_queries(self, layer: int, Q: int, nq: int, device=None) -> torch.Tensor:
        """[Q*nq, d_in] query-token vectors from the key distribution (they go through the key SAE,
        which is the shared codebook)."""
        cfg = self.cfg
        device = self.device if device is None else device
        return G.activations(cfg.seed + 900001, layer, 0, Q * nq, cfg.key.d_in, cfg.dtype, self._scale,
                             device, tid=G.TID_QUERY_X)
