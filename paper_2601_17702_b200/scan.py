"""Host driver loop of the streaming scan (Algorithm 1, Phase 1): per context chunk and target layer,
encode the transient key (and optionally query) projections, build the chunk's CSR postings and hand
them to the host-resident index. It only sequences calls of the C ABI on torch-owned buffers; device
memory is allocated once, for one chunk, and reused for every chunk of the context."""
from __future__ import annotations

import contextlib

import torch

from . import binding as B


# "auto" grouping: the layers of an SAE stream share one launch when the encoder's input is this narrow (the launch is
# then bound by the Top-k filter, and a grouped launch keeps every SM busy to its end). Wider encoders are bound by the
# operand feed and the power cap; there a launch whose CTA pairs all walk ONE encoder's weights in step is faster
# (measured on the 4096 -> 32768 query encoders: four layers in one launch take 14 % longer than four launches).
AUTO_GROUP_MAX_D_IN = 1024


class SaeSlot:
    """One SAE stream of the scan (e.g. 'key' or 'query'): per-layer encoders plus the chunk-sized
    device buffers its outputs go through."""

    def __init__(self, name: str, saes: list[B.Sae], k: int, chunk: int, with_values: bool = False):
        self.name, self.saes, self.k, self.chunk = name, saes, k, chunk
        dev = saes[0].W_enc.device
        self.d_sae = saes[0].d_sae
        n_layers = len(saes)
        self.ids = [torch.empty((chunk, k), dtype=torch.int32, device=dev) for _ in range(n_layers)]
        self.vals = [torch.empty((chunk, k), dtype=torch.float32, device=dev) for _ in range(n_layers)]
        self.row_ptr = [torch.zeros(self.d_sae + 1, dtype=torch.int32, device=dev) for _ in range(n_layers)]
        self.pos = [torch.zeros(chunk * k, dtype=torch.int32, device=dev) for _ in range(n_layers)]
        self.pval = [torch.zeros(chunk * k, dtype=torch.float32, device=dev) for _ in range(n_layers)] if with_values else None
        self.ws = B.new_workspace(max(s.encode_workspace_bytes(chunk, k) for s in saes), dev)
        self.index = B.Index(n_layers, self.d_sae)


class ScanPipeline:
    def __init__(self, slots: list[SaeSlot], grouped: bool | str = "auto", overlap: bool = False):
        """grouped: how the encodes of a chunk are launched (bf16 encoders; fp32 ones always go one by one).
        True / "all": the layers of all SAE streams in grouped launches (one persistent kernel per up to
        S3_MAX_ENCODE_ITEMS encoders); "slot": one grouped launch per SAE stream; a stream's name (e.g. "key"): only
        that stream's layers are grouped; False / "none": one launch pair per encoder; "auto" (default): per stream,
        grouped when the encoder input is at most AUTO_GROUP_MAX_D_IN wide.
        overlap: when a chunk has both wide encoders (launched one by one, each leaving some SMs without a work unit) and
        a grouped launch of narrow ones, the grouped launch runs on a second stream, limited to the SMs the wide launches
        leave free, so that it proceeds beside them instead of after them. Off by default: measured on the 128K-token
        workload the four key encoders then take the whole window of the query launches on the 10 free CTA pairs (8.3 ms
        instead of 1.3 ms alone) while each query launch runs 6 % slower beside them, and the step gets no shorter."""
        self.slots = slots
        self.n_layers = len(slots[0].saes)
        self.overlap = overlap
        self.side = None           # second stream of the overlapped grouped launch
        mode = {True: "all", False: "none"}.get(grouped, grouped)
        if not all(sae.dtype == B.S3_BF16 for s in slots for sae in s.saes):
            mode = "none"
        self.auto = mode == "auto"
        self.group_mode = mode
        self.ws_enc = None         # workspace of the grouped encode, sized at the first chunk
        n_post = sum(B.s3_postings_workspace_bytes(s.chunk, s.k, s.d_sae) for s in slots) * self.n_layers
        self.ws_post = B.new_workspace(n_post, slots[0].ids[0].device)
        self.launches = 0          # kernels of this library enqueued so far
        self.timers = None         # when set to a dict: name -> list of (start, end) CUDA events around each call
        self.host_syncs = 0        # host-blocking calls made by scan_chunk (none: ordering is by stream and events)

    @contextlib.contextmanager
    def _timed(self, name: str):
        if self.timers is None:
            yield
            return
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        yield
        e1.record()
        self.timers.setdefault(name, []).append((e0, e1))

    def reserve_index(self, n_tokens: int):
        for s in self.slots:
            per_layer = n_tokens * s.k * (8 if s.pval else 4) + (n_tokens // s.chunk + 2) * (s.d_sae + 1 + 64) * 4
            s.index.reserve(per_layer * self.n_layers + (1 << 20))

    def scan_chunk(self, pos_base: int, x_by_slot: dict[str, list[torch.Tensor]], append: bool = True):
        """x_by_slot[name][layer] is the [T, d_in] projection of this chunk for that SAE stream. append=False leaves
        out the hand-over to the host index (to time the device work without the copies)."""
        items = []
        enc_items = []
        singles = []
        T = None
        for s in self.slots:
            xs = x_by_slot[s.name]
            for l in range(self.n_layers):
                x = xs[l]
                T = x.shape[0]
                if self.group_mode in ("all", "slot", s.name) or (self.auto and s.saes[l].d_in <= AUTO_GROUP_MAX_D_IN):
                    enc_items.append((s.name, B.make_encode_item(s.saes[l], x, s.k, s.ids[l][:T], s.vals[l][:T])))
                else:
                    singles.append((s, l, x))
                items.append(B.make_postings_item(s.ids[l][:T], s.d_sae, pos_base, s.row_ptr[l], s.pos[l],
                                                  s.vals[l][:T] if s.pval else None, s.pval[l] if s.pval else None))
        groups = []
        for name, item in enc_items:
            new_group = not groups or len(groups[-1][1]) == B.S3_MAX_ENCODE_ITEMS or (self.group_mode != "all" and groups[-1][0] != name)
            if new_group:
                groups.append((name, []))
            groups[-1][1].append(item)
        need = max((B.s3_sae_encode_grouped_workspace_bytes(g) for _, g in groups), default=0)
        if groups and (self.ws_enc is None or self.ws_enc.numel() < need):
            assert self.ws_enc is None, "the grouped-encode workspace is sized by the first (full) chunk"
            self.ws_enc = B.new_workspace(need, self.slots[0].ids[0].device)

        # SMs the wide launches leave without a work unit: the grouped launch of the narrow encoders can have them
        free_ctas = 0
        if self.overlap and groups and singles:
            n_sm = torch.cuda.get_device_properties(self.slots[0].ids[0].device).multi_processor_count
            free_ctas = min(n_sm - B.s3_sae_encode_ctas(s.saes[l], x.shape[0]) for s, l, x in singles)
        main = torch.cuda.current_stream()
        if free_ctas >= 2:
            if self.side is None:
                self.side = torch.cuda.Stream(device=self.slots[0].ids[0].device)
            self.side.wait_stream(main)          # the chunk's inputs, and the previous chunk's postings that read ids, are done
        for s, l, x in singles:
            with self._timed("encode_" + s.name):
                B.s3_sae_encode_topk(s.saes[l], x, s.k, s.ids[l][:x.shape[0]], s.vals[l][:x.shape[0]], s.ws)
            self.launches += 2
        with torch.cuda.stream(self.side if free_ctas >= 2 else main):
            for name, group in groups:
                with self._timed("encode_group" if self.group_mode == "all" else "encode_group_" + name):
                    B.s3_sae_encode_topk_grouped(group, self.ws_enc, free_ctas if free_ctas >= 2 else 0)
                self.launches += 2         # persistent encode over all items, selection over all items
        if free_ctas >= 2:
            main.wait_stream(self.side)
        # the previous chunk's device->host copies read row_ptr/pos: order the overwrite after them
        for s in self.slots:
            s.index.stream_wait()
        for i in range(0, len(items), 32):
            with self._timed("postings"):
                B.s3_postings_build_batched(items[i:i + 32], self.ws_post)
            self.launches += 2         # partition by bucket, bucket sort
        if not append:
            return
        for s in self.slots:
            for l in range(self.n_layers):
                s.index.append(l, s.row_ptr[l], s.pos[l], T, s.k, pos_base, s.pval[l] if s.pval else None)

    def finish(self):
        for s in self.slots:
            s.index.sync()
            code = B.s3_workspace_status(s.ws)
            assert code == 0
        if self.ws_enc is not None:
            assert B.s3_workspace_status(self.ws_enc) == 0
        assert B.s3_workspace_status(self.ws_post) == 0

    def close(self):
        for s in self.slots:
            s.index.close()


def stage_index_on_device(index: B.Index, device) -> list[tuple[torch.Tensor, torch.Tensor]]:
    """Merged per-layer CSRs of a host index, uploaded for retrieval."""
    out = []
    for l in range(index.n_layers):
        rp, ps, _ = index.export_csr(l)
        if ps.numel() == 0:
            ps = torch.zeros(1, dtype=torch.int32)
        out.append((rp.to(device), ps.to(device)))
    return out
