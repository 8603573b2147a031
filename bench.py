#!/usr/bin/env python
"""Benchmark of the select + compact + KV-compaction path.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

One "step" is one pass of the whole path over one batch of synthetic input:
civic_select_seq (selection and sequence-level indices, one launch) -> civic_compact (hidden +
position ids) -> civic_compact_kv (all layers, K and V).  The default workload is the
Qwen3-VL-8B-shaped K/V compaction configuration (16 sequences x 1088 tokens, 36 layers), with
the batch's hidden states and position ids included so that every step of the path runs.

Prints ONE JSON line (rank 0).  `value` is whole-job compacted GB/s with inputs resident in
HBM: the bytes the method has to move (every kept row read once and written once, plus
scores in and indices out) divided by the device time of a step.  With N > 1 every rank
compacts its own batch (no data-path collective; weak scaling) and the line reports the sum.
"""

from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "compacted_GBps_select_compact_kv"
UNIT = "GB/s"
KV_EVENT_STRIDE = 10
FALLBACK_HBM_GBS = 6650.0  # earlier measurement on this machine, used when MEASURED_PEAKS.json is absent

# DRAM bytes (read + write) of ONE civic_compact_kv launch, keyed by workload name: NOT measured by
# the run that prints them, but taken from the ncu captures summarised in profiles/ (an 8-layer case
# of the same kernel, dram__bytes_read.sum + dram__bytes_write.sum per launch).  Scaled to the full
# launch as: reads x layers / 8 (they grow in proportion to the layers), writes = algorithmic bytes
# written minus what is still dirty in L2 when the kernel ends (55 .. 57 MB, a property of L2, not of
# the layer count).  Absent = not captured for that workload.
NCU_DRAM_TRAFFIC_PER_LAUNCH = {
    "c3_kv_qwen3vl8b": (1_856_400_000, "profiles/gather_rows_kernel_c3_kv.md"),
    "c5_hires_keep_1_2": (1_794_800_000, "profiles/gather_rows_kernel_layouts_c3_c5.md"),
    "c5_hires_keep_1_3": (1_176_900_000, "profiles/gather_rows_kernel_layouts_c3_c5.md"),
    "c5_hires_keep_1_4": (868_200_000, "profiles/gather_rows_kernel_layouts_c3_c5.md"),
}
TRAFFIC_SOURCE = ("ncu capture of an 8-layer case of the same kernel, scaled to {layers} layers; "
                  "not measured by this run ({file})")


def ncu_traffic(wl_name, layers):
    """(bytes per launch, where the figure comes from) or (None, None)."""
    hit = NCU_DRAM_TRAFFIC_PER_LAUNCH.get(wl_name)
    if not hit:
        return None, None
    return hit[0], TRAFFIC_SOURCE.format(layers=layers, file=hit[1])


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--workload", default="c3_kv_qwen3vl8b")
    ap.add_argument("--impl", default="civic", choices=["civic", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--kv-layout", default="token_major", choices=["token_major", "head_major", "paged"],
                    help="K/V cache layout: [seq, token, heads*dim] rows (default), [seq, head, token, dim] "
                         "pieces, or token-major sources into a paged cache of 16-token pages")
    ap.add_argument("--merge", action="store_true",
                    help="also build the compact prefill sequence (Eq. 13 merge of text and kept visual "
                         "rows) and its plane-major position ids in every step")
    ap.add_argument("--graph", action="store_true",
                    help="capture one step in a CUDA graph and time its replays: the GPU-side latency of the "
                         "step without the Python binding's per-call host time (for the small workloads)")
    ap.add_argument("--no-others", action="store_true",
                    help="skip the other workloads that the default run times after the main one")
    ap.add_argument("--layers", type=int, default=0,
                    help="shrink the workload to this many K/V layers (profiling a small case); "
                         "the JSON line then names the reduced workload")
    return ap.parse_args()


def step_bytes(wl, merge=False):
    """Algorithmic bytes of one step, by part."""
    from paper_2605_28115_b200 import workloads as W

    kv = W.kv_algorithmic_bytes(wl)
    hidden = 2 * wl.n_seg * wl.k * wl.hidden_row_bytes if wl.hidden_dim else 0
    pos = 2 * wl.n_seg * wl.k * 12
    select = wl.n_seg * wl.n * 4 + wl.n_seg * wl.k * 4
    seq = (wl.n_seg * wl.k * 4 + wl.n_seg * wl.s_out * 4) if wl.n_layers else 0
    out = {"kv": kv, "hidden": hidden, "pos": pos, "select": select, "seq_idx": seq}
    if merge:  # every row of the compact sequence read once and written once; 3 planes of pos ids
        out["merge"] = 2 * wl.n_seg * wl.s_out * wl.hidden_row_bytes
        out["pos_planes"] = 2 * 3 * wl.n_seg * wl.s_out * 4
    out["total"] = sum(out.values())
    return out


def pick_workload(args):
    from paper_2605_28115_b200 import workloads as W

    wl = W.BY_NAME[args.workload]
    if args.layers and wl.n_layers:
        wl = wl.replace(name=f"{wl.name}_reduced_to_{args.layers}_layers", n_layers=args.layers)
    return wl


def parallelism_of(world):
    return f"dp{world}" if world > 1 else "single"


def config_of(wl, extra=None):
    cfg = {"workload": wl.name, "n_seg": wl.n_seg, "grid_thw": [wl.t, wl.h, wl.w],
           "region_hw": [wl.region_h, wl.region_w], "floor_per_region": wl.floor_m, "k": wl.k,
           "scores": wl.score_kind, "hidden_dim": wl.hidden_dim, "layers": wl.n_layers,
           "kv_row_bytes": wl.kv_row_bytes, "seq_len": wl.seq_len, "s_out": wl.s_out,
           "text_tokens": [wl.text_before, wl.text_after],
           "l2": ("inputs larger than L2: each step streams the whole K/V set through it, no flush" if wl.n_layers
                  else "working set smaller than L2 and not flushed: a latency figure, not a bandwidth figure")}
    if extra:
        cfg.update(extra)
    return cfg


def measured_tensor_peak():
    """(burst, sustained) dense bf16 TFLOP/s of this machine's B200s and where they come from."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            d = json.load(f)
        return float(d["bf16_tflops"]), float(d["bf16_tflops_sustained"]), "measured (MEASURED_PEAKS.json)"
    except Exception:
        return 1590.0, 1400.0, "fallback (1.59 PFLOP/s burst, 1.4 sustained: earlier measurement)"


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback (6.65 TB/s, earlier measurement on this pool)"


# ----------------------------------------------------------------------------- clocks

class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU through NVML (read-only) while the
    timed region runs."""

    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown",
               0x4: "sw_power_cap", 0x80: "hw_power_brake_slowdown", 0x2: "applications_clocks_setting",
               0x100: "display_clock_setting", 0x10: "sync_boost"}

    def __init__(self, torch_device_index: int, period_s: float = 0.02):
        self.period = period_s
        self.samples = []
        self.reason_bits = 0
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        self.error = None
        try:
            import pynvml
            import torch

            pynvml.nvmlInit()
            self.nv = pynvml
            uuid = str(torch.cuda.get_device_properties(torch_device_index).uuid)
            if not uuid.startswith("GPU-"):
                uuid = "GPU-" + uuid
            try:
                self.handle = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode())
            except Exception:
                self.handle = pynvml.nvmlDeviceGetHandleByUUID(uuid)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.handle, pynvml.NVML_CLOCK_SM))
        except Exception as e:  # pragma: no cover - depends on the box
            self.error = repr(e)
            self.nv = None

    def _run(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.handle, nv.NVML_CLOCK_SM)))
                self.reason_bits |= int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.handle))
            except Exception as e:  # pragma: no cover
                self.error = repr(e)
                return
            self._stop.wait(self.period)

    def start(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()
        out = {"sm_mhz": int(statistics.median(self.samples)) if self.samples else None,
               "sm_max_mhz": self.max_mhz, "samples": len(self.samples),
               "reasons": sorted(name for bit, name in self.REASONS.items() if self.reason_bits & bit)}
        if self.error:
            out["error"] = self.error
        return out


# ----------------------------------------------------------------------------- CUDA arm

class DeviceState:
    """Inputs and outputs of one rank, resident on its GPU."""

    PAGE = 16

    def __init__(self, wl, dev, rank, kv_layout="token_major", merge=False):
        import torch

        from paper_2605_28115_b200 import civic
        from paper_2605_28115_b200 import workloads as W

        self.wl, self.dev = wl, dev
        self.kv_layout, self.merge = kv_layout, merge and bool(wl.hidden_dim) and bool(wl.n_layers)
        wl_r = wl.replace(config_id=wl.config_id + 100 * rank) if rank else wl  # per-rank seeds
        self.scores_host = W.scores(wl_r)
        self.pos_host = W.pos_ids(wl)
        self.scores = torch.from_numpy(self.scores_host).to(dev)
        self.pos = torch.from_numpy(self.pos_host).to(dev)
        self.hidden = W.hidden(wl_r, dev) if wl.hidden_dim else None
        self.desc = civic.SelectDesc(wl.t, wl.h, wl.w, wl.region_h, wl.region_w, wl.floor_m, wl.k)
        self.keep = torch.empty((wl.n_seg, wl.k), dtype=torch.int32, device=dev)
        self.hidden_out = (torch.empty((wl.n_seg, wl.k, wl.hidden_dim), dtype=torch.bfloat16, device=dev)
                           if wl.hidden_dim else None)
        self.pos_out = torch.empty((wl.n_seg, wl.k, 3), dtype=torch.int32, device=dev)
        self.seq_idx = torch.empty((wl.n_seg, wl.s_out), dtype=torch.int32, device=dev)
        self.k_src = [W.kv_layer(wl_r, l, 0, dev) for l in range(wl.n_layers)]
        self.v_src = [W.kv_layer(wl_r, l, 1, dev) for l in range(wl.n_layers)]
        self.block_table = None
        if kv_layout == "head_major":  # the same seeded payload read as [seq, head, token, dim]
            self.k_src = [x.view(wl.n_seg, wl.kv_heads, wl.seq_len, wl.head_dim) for x in self.k_src]
            self.v_src = [x.view(wl.n_seg, wl.kv_heads, wl.seq_len, wl.head_dim) for x in self.v_src]
            shape = (wl.n_seg, wl.kv_heads, wl.s_out, wl.head_dim)
        elif kv_layout == "paged":  # every sequence owns ceil(s_out / PAGE) pages of a shuffled pool
            per_seq = -(-wl.s_out // self.PAGE)
            g = torch.Generator(device="cpu")
            g.manual_seed(wl.seed + 900 + rank)
            self.block_table = torch.randperm(wl.n_seg * per_seq, generator=g).to(torch.int32) \
                .view(wl.n_seg, per_seq).contiguous().to(dev)
            shape = (wl.n_seg * per_seq, self.PAGE, wl.kv_heads, wl.head_dim)
        else:
            shape = (wl.n_seg, wl.s_out, wl.kv_heads, wl.head_dim)
        self.k_dst = [torch.empty(shape, dtype=torch.bfloat16, device=dev) for _ in range(wl.n_layers)]
        self.v_dst = [torch.empty(shape, dtype=torch.bfloat16, device=dev) for _ in range(wl.n_layers)]
        make = {"token_major": civic.kv_tables, "head_major": civic.kv_heads_tables,
                "paged": civic.kv_paged_tables}[kv_layout]
        self.tables = make(self.k_src, self.v_src, self.k_dst, self.v_dst) if wl.n_layers else None
        if self.merge:
            self.text = W.payload_bf16((wl.n_seg, wl.seq_len, wl.hidden_dim), wl_r.seed + 700, dev)
            self.merged = torch.empty((wl.n_seg, wl.s_out, wl.hidden_dim), dtype=torch.bfloat16, device=dev)
            planes = torch.arange(wl.seq_len, dtype=torch.int32).repeat(3, wl.n_seg, 1)
            vis = torch.from_numpy(self.pos_host).permute(2, 0, 1) + wl.text_before  # (t,h,w) planes
            planes[:, :, wl.text_before:wl.text_before + wl.n] = vis
            self.pos_planes = planes.contiguous().to(dev)
            self.pos_planes_out = torch.empty((3, wl.n_seg, wl.s_out), dtype=torch.int32, device=dev)

    def compact_kv(self):
        from paper_2605_28115_b200 import civic

        if self.kv_layout == "head_major":
            civic.civic_compact_kv_heads(self.tables, self.seq_idx)
        elif self.kv_layout == "paged":
            civic.civic_compact_kv_paged(self.tables, self.seq_idx, self.block_table)
        else:
            civic.civic_compact_kv(self.tables, self.seq_idx)

    def step(self, kv_events=None):
        """One pass of the whole path on the current stream (asynchronous)."""
        from paper_2605_28115_b200 import civic

        wl = self.wl
        if self.tables is not None:
            civic.civic_select_seq(self.scores, self.desc, wl.seq_len, wl.text_before,
                                   keep_idx=self.keep, seq_idx=self.seq_idx)
        else:
            civic.civic_select(self.scores, self.desc, keep_idx=self.keep)
        civic.civic_compact(self.hidden, self.pos, self.keep, hidden_out=self.hidden_out, pos_out=self.pos_out)
        if self.merge:
            civic.civic_merge_embeddings(self.text, self.hidden, self.keep, wl.text_before, merged=self.merged)
            civic.civic_compact_pos_planes(self.pos_planes, self.seq_idx, pos_out=self.pos_planes_out)
        if self.tables is not None:
            if kv_events is not None:
                kv_events[0].record()
            self.compact_kv()
            if kv_events is not None:
                kv_events[1].record()


class HostState:
    """Pinned host copies of one rank's inputs and result buffers for the end-to-end number.

    mode "zero_copy": the big payloads (hidden, K/V) stay in pinned host memory and their
    pointers go straight into the C-ABI calls: the kernels read only the KEPT rows over PCIe and
    write the compacted rows straight back to pinned host memory.  Only scores and position ids
    (small) are copied to the device, and the index results copied back.
    mode "staged": every input is copied to the device, the path runs on device buffers, every
    result is copied back.
    mode "pipelined": the K/V kernel reads the kept rows from pinned host memory (as in zero_copy) but
    writes them into device buffers, a few layers per launch; a second stream's copy engine moves each
    finished chunk to pinned host memory while the kernel reads the next one.  PCIe then carries the
    kernel's read requests and completions in one direction pair and plain bulk writes in the other.
    """

    CHUNK_LAYERS = 2

    def __init__(self, st: DeviceState, mode: str):
        import torch

        from paper_2605_28115_b200 import civic

        pin = lambda x: torch.empty(x.shape, dtype=x.dtype, device="cpu", pin_memory=True).copy_(x)
        empty = lambda x: torch.empty(x.shape, dtype=x.dtype, device="cpu", pin_memory=True)
        size = lambda x: x.numel() * x.element_size()
        self.st, self.mode = st, mode
        wl = st.wl
        self.small_in = [(pin(st.scores), st.scores), (pin(st.pos), st.pos)]
        self.small_out = [(st.keep, empty(st.keep)), (st.pos_out, empty(st.pos_out))]
        self.hidden_h = pin(st.hidden) if st.hidden is not None else None
        self.hidden_out_h = empty(st.hidden_out) if st.hidden_out is not None else None
        self.k_src_h = [pin(x) for x in st.k_src]
        self.v_src_h = [pin(x) for x in st.v_src]
        self.k_dst_h = [empty(x) for x in st.k_dst]
        self.v_dst_h = [empty(x) for x in st.v_dst]
        small_in = sum(size(h) for h, _ in self.small_in)
        small_out = sum(size(h) for _, h in self.small_out)
        big_out = sum(size(x) for x in self.k_dst_h + self.v_dst_h) + \
            (size(self.hidden_out_h) if self.hidden_out_h is not None else 0)
        if mode == "zero_copy":
            self.tables = (civic.kv_tables(self.k_src_h, self.v_src_h, self.k_dst_h, self.v_dst_h)
                           if wl.n_layers else None)
            # bytes that cross PCIe towards the device: small inputs + the kept rows the kernels read
            self.h2d_bytes = small_in + big_out
        elif mode == "pipelined":
            c = self.CHUNK_LAYERS
            self.chunks = [range(l, min(l + c, wl.n_layers)) for l in range(0, wl.n_layers, c)]
            self.chunk_tables = [civic.kv_tables([self.k_src_h[l] for l in ls], [self.v_src_h[l] for l in ls],
                                                 [st.k_dst[l] for l in ls], [st.v_dst[l] for l in ls])
                                 for ls in self.chunks]
            self.copy_stream = torch.cuda.Stream()
            self.gathered = [torch.cuda.Event() for _ in self.chunks]
            self.drained = [torch.cuda.Event() for _ in self.chunks]
            self.first = True
            self.h2d_bytes = small_in + big_out
        else:
            self.h2d_bytes = small_in + sum(size(x) for x in self.k_src_h + self.v_src_h) + \
                (size(self.hidden_h) if self.hidden_h is not None else 0)
        self.d2h_bytes = small_out + big_out

    def step(self):
        from paper_2605_28115_b200 import civic

        st, wl = self.st, self.st.wl
        for h, d in self.small_in:
            d.copy_(h, non_blocking=True)
        if self.mode == "zero_copy":
            if self.tables is not None:
                civic.civic_select_seq(st.scores, st.desc, wl.seq_len, wl.text_before,
                                       keep_idx=st.keep, seq_idx=st.seq_idx)
            else:
                civic.civic_select(st.scores, st.desc, keep_idx=st.keep)
            civic.civic_compact(self.hidden_h, st.pos, st.keep, hidden_out=self.hidden_out_h,
                                pos_out=st.pos_out)
            if self.tables is not None:
                civic.civic_compact_kv(self.tables, st.seq_idx)
        elif self.mode == "pipelined":
            import torch

            main = torch.cuda.current_stream()
            civic.civic_select_seq(st.scores, st.desc, wl.seq_len, wl.text_before, keep_idx=st.keep, seq_idx=st.seq_idx)
            civic.civic_compact(self.hidden_h, st.pos, st.keep, hidden_out=self.hidden_out_h, pos_out=st.pos_out)
            for c, ls in enumerate(self.chunks):
                if not self.first:
                    main.wait_event(self.drained[c])  # the previous step's copy of this chunk has left the buffers
                civic.civic_compact_kv(self.chunk_tables[c], st.seq_idx)
                self.gathered[c].record(main)
                with torch.cuda.stream(self.copy_stream):
                    self.copy_stream.wait_event(self.gathered[c])
                    for l in ls:
                        self.k_dst_h[l].copy_(st.k_dst[l], non_blocking=True)
                        self.v_dst_h[l].copy_(st.v_dst[l], non_blocking=True)
                    self.drained[c].record(self.copy_stream)
            self.first = False
            main.wait_stream(self.copy_stream)
        else:
            if self.hidden_h is not None:
                st.hidden.copy_(self.hidden_h, non_blocking=True)
            for h, d in zip(self.k_src_h + self.v_src_h, st.k_src + st.v_src):
                d.copy_(h, non_blocking=True)
            st.step()
            if self.hidden_out_h is not None:
                self.hidden_out_h.copy_(st.hidden_out, non_blocking=True)
            for d, h in zip(st.k_dst + st.v_dst, self.k_dst_h + self.v_dst_h):
                h.copy_(d, non_blocking=True)
        for d, h in self.small_out:
            h.copy_(d, non_blocking=True)

    def matches_device_results(self) -> bool:
        """After a device-resident step and a host step: the host buffers hold the same bytes."""
        import torch

        st = self.st
        pairs = list(zip(st.k_dst + st.v_dst, self.k_dst_h + self.v_dst_h))
        if st.hidden_out is not None:
            pairs.append((st.hidden_out, self.hidden_out_h))
        pairs += self.small_out
        return all(torch.equal(d.cpu(), h) for d, h in pairs)


def cpu_baseline(st: DeviceState, limit_s: float = 20.0):
    """The oracle as it stands, timed on this machine's host cores on the same inputs (copied
    from the device): a few whole passes, bounded by `limit_s`."""
    import numpy as np
    import torch

    import oracle

    wl = st.wl
    o = oracle.default
    threads = o.set_threads(0)
    bits = lambda x: x.contiguous().view(torch.int16).cpu().numpy()
    n_layers = wl.n_layers
    row = wl.kv_heads * wl.head_dim
    ks = [bits(x).reshape(wl.n_seg, -1, row) for x in st.k_src[:n_layers]]
    vs = [bits(x).reshape(wl.n_seg, -1, row) for x in st.v_src[:n_layers]]
    hidden = bits(st.hidden) if st.hidden is not None else None
    sample = wl.replace(n_layers=n_layers)
    nbytes = step_bytes(sample)["total"]
    times = []
    t_begin = time.perf_counter()
    while len(times) < 3 or (time.perf_counter() - t_begin < limit_s / 2 and len(times) < 15):
        t0 = time.perf_counter()
        keep = o.select(st.scores_host, wl.t, wl.h, wl.w, wl.region_h, wl.region_w, wl.floor_m, wl.k)
        o.compact(hidden, st.pos_host, keep)
        if n_layers:
            idx = o.seq_indices(keep, wl.seq_len, wl.text_before, wl.n)
            o.compact_kv(ks, vs, idx)
        times.append(time.perf_counter() - t0)
    med = statistics.median(times)
    return {"value": nbytes / med / 1e9, "unit": UNIT, "cores": threads, "kind": "oracle",
            "sample": f"whole path on {wl.n_seg} segments with all {n_layers} K/V layers, "
                      f"median of {len(times)} runs, {med * 1e3:.1f} ms per run",
            "ms_per_sample": med * 1e3}


def path_equals_oracle(st: DeviceState) -> bool:
    """Every result of the last device-resident step of `st` against the CPU oracle, bit for bit:
    keep indices, hidden rows, position ids, sequence indices, all layers' K and V rows."""
    import numpy as np
    import torch

    import oracle

    wl, o = st.wl, oracle.default
    o.set_threads(0)
    bits = lambda x: x.contiguous().view(torch.int16).cpu().numpy()
    keep = o.select(st.scores_host, wl.t, wl.h, wl.w, wl.region_h, wl.region_w, wl.floor_m, wl.k)
    ok = np.array_equal(st.keep.cpu().numpy(), keep)
    h_o, p_o = o.compact(bits(st.hidden) if st.hidden is not None else None, st.pos_host, keep)
    if st.hidden is not None:
        ok = ok and np.array_equal(bits(st.hidden_out), h_o)
    ok = ok and np.array_equal(st.pos_out.cpu().numpy(), p_o)
    if wl.n_layers and st.kv_layout == "token_major":
        idx = o.seq_indices(keep, wl.seq_len, wl.text_before, wl.n)
        ok = ok and np.array_equal(st.seq_idx.cpu().numpy(), idx)
        row = wl.kv_heads * wl.head_dim
        flat = lambda x: bits(x).reshape(wl.n_seg, -1, row)
        for l0 in range(0, wl.n_layers, 6):  # six layers at a time bounds the host copies
            ls = range(l0, min(l0 + 6, wl.n_layers))
            k_o, v_o = o.compact_kv([flat(st.k_src[l]) for l in ls], [flat(st.v_src[l]) for l in ls], idx)
            for j, l in enumerate(ls):
                ok = ok and np.array_equal(flat(st.k_dst[l]), k_o[j]) and np.array_equal(flat(st.v_dst[l]), v_o[j])
    return bool(ok)


def contiguous_copy_rate(st: DeviceState, launches=10):
    """GB/s of civic_compact_kv when it keeps EVERY row (identity indices): the same kernel as a plain
    contiguous copy of the whole K/V set, i.e. the most this gather could reach on this GPU today."""
    import torch

    from paper_2605_28115_b200 import civic

    wl = st.wl
    idx = torch.arange(wl.seq_len, dtype=torch.int32, device=st.dev).repeat(wl.n_seg, 1).contiguous()
    k_all = [torch.empty_like(x) for x in st.k_src]
    v_all = [torch.empty_like(x) for x in st.v_src]
    tables = civic.kv_tables(st.k_src, st.v_src, k_all, v_all)
    for _ in range(2):
        civic.civic_compact_kv(tables, idx)
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    start.record()
    for _ in range(launches):
        civic.civic_compact_kv(tables, idx)
    end.record()
    torch.cuda.synchronize()
    nbytes = 2 * sum(x.numel() * x.element_size() for x in st.k_src + st.v_src)
    return nbytes / (start.elapsed_time(end) / launches * 1e-3) / 1e9


def index_check_cost(st: DeviceState, launches=20):
    """Microseconds per civic_compact_kv launch with the device-side index validation switched on
    (the checked kernels: every index tested against its range, faults recorded, nothing trapped)."""
    import torch

    from paper_2605_28115_b200 import civic

    record = torch.zeros(4, dtype=torch.int32, device=st.dev)
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with civic.index_check(record):
        for _ in range(3):
            st.compact_kv()
        torch.cuda.synchronize()
        start.record()
        for _ in range(launches):
            st.compact_kv()
        end.record()
        torch.cuda.synchronize()
    return {"us_per_launch": start.elapsed_time(end) / launches * 1e3, "fault_record": record.cpu().tolist()}


def kv_roofline(wl, kv_bytes, kv_ms, kv_layout="token_major", default_variant=True):
    """The roofline object of the K/V gather from event-bracketed launches (ms each)."""
    kv_avg = sum(kv_ms) / len(kv_ms)
    peak, which = measured_peak()
    achieved = kv_bytes / (kv_avg * 1e-3) / 1e9
    kernel = {"token_major": "civic_compact_kv", "head_major": "civic_compact_kv_heads",
              "paged": "civic_compact_kv_paged"}[kv_layout]
    traffic, source = ncu_traffic(wl.name, wl.n_layers) if default_variant else (None, None)
    return {"bound": "hbm", "kernel": kernel, "achieved": achieved, "peak": peak, "unit": "GB/s",
            "frac": achieved / peak, "peak_source": which, "traffic": traffic, "traffic_source": source,
            "algorithmic_bytes_per_launch": kv_bytes, "us_per_launch": kv_avg * 1e3,
            "us_per_launch_min": min(kv_ms) * 1e3, "launches_timed": len(kv_ms),
            "frac_of_8TBps_nominal": achieved / 8000.0}


def time_other_path_workload(wl, dev, steps, with_oracle):
    """One of the other select + compact (+ K/V) configurations on one GPU: device-resident steps as a
    plain loop; the K/V configurations bracket every tenth K/V launch with events, the small ones are
    also timed as replays of a CUDA graph of one step."""
    import torch

    from paper_2605_28115_b200 import civic

    st = DeviceState(wl, dev, 0)
    nbytes = step_bytes(wl)
    for _ in range(5):
        st.step()
    torch.cuda.synchronize()
    kv_ev = {i: (torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
             for i in range(0, steps, 10)} if wl.n_layers else {}
    sampler = ClockSampler(torch.device(dev).index or 0)
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    launches0 = civic.launch_count()
    sampler.start()
    torch.cuda.synchronize()
    start.record()
    for i in range(steps):
        st.step(kv_ev.get(i))
    end.record()
    torch.cuda.synchronize()
    ms = start.elapsed_time(end) / steps
    out = {"workload": wl.name, "steps": steps, "us_per_step": ms * 1e3,
           "value": nbytes["total"] / (ms * 1e-3) / 1e9, "unit": UNIT, "bytes_per_step": nbytes["total"],
           "gpu_launches": civic.launch_count() - launches0,
           "l2": config_of(wl)["l2"]}
    if kv_ev:
        out["roofline"] = kv_roofline(wl, nbytes["kv"], [a.elapsed_time(b) for a, b in kv_ev.values()])
    else:  # launch-bound: also as a graph of one step, without the binding's host time per call
        side = torch.cuda.Stream()
        with torch.cuda.stream(side):
            st.step()
            torch.cuda.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=side):
                st.step()
        for _ in range(5):
            graph.replay()
        torch.cuda.synchronize()
        start.record()
        for _ in range(steps):
            graph.replay()
        end.record()
        torch.cuda.synchronize()
        out["graph_replay_us_per_step"] = start.elapsed_time(end) / steps * 1e3
        # a replay has a floor of its own (about 8 us here, whatever the graph holds): 20 steps per graph
        with torch.cuda.stream(side):
            graph20 = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph20, stream=side):
                for _ in range(20):
                    st.step()
        out["graph_of_20_steps_us_per_step"] = time_loop(graph20.replay, max(steps // 20, 20), 3) / 20
        peak, _ = measured_peak()
        out["hbm_time_us_at_measured_peak"] = nbytes["total"] / peak / 1e3
        st.step()
        torch.cuda.synchronize()
    out["clocks"] = sampler.stop()
    if with_oracle:
        out["equals_oracle"] = path_equals_oracle(st)
    return out


def time_loop(step, steps, warm):
    """Microseconds per call of `step` (CUDA events on the current stream, after `warm` calls)."""
    import torch

    for _ in range(warm):
        step()
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    start.record()
    for _ in range(steps):
        step()
    end.record()
    torch.cuda.synchronize()
    return start.elapsed_time(end) / steps * 1e3


def aggregate_within_bound(x0, anchors, tau, z0, mass):
    """Image 0 of a civic_anchor_aggregate result against the fp64 oracle: the largest error as a
    share of the element-wise bound derived from the arithmetic (bf16 anchors, fp32 accumulation,
    bf16 weights and result), and the oracle's time."""
    import numpy as np

    from oracle import aggregate as OA

    d_v = x0.shape[2]
    x64, a64 = x0[0].double().cpu().numpy(), anchors.double().cpu().numpy()
    t0 = time.perf_counter()
    z_o, w_o = OA.anchor_aggregate(x64, a64, tau)
    seconds = time.perf_counter() - t0
    d_cos = 2.0 ** -9 + d_v * 2.0 ** -24
    eps_w = np.expm1(2 * d_cos / tau) + 2.0 ** -8
    w = OA.aggregation_weights(x64, a64, tau)
    bound = eps_w * (w @ np.abs(x64)) + 2.0 ** -9 * np.abs(z_o)
    err = np.abs(z0[0].float().cpu().numpy().astype(np.float64) - z_o)
    share = float(np.max(err / np.maximum(bound, 1e-300)))
    mass_o = w.sum(axis=0)
    share = max(share, float(np.max(np.abs(mass[0].cpu().numpy() - mass_o) / (eps_w * mass_o + 1e-30))))
    return share, float(err.max()), seconds


def time_aggregate(w, dev, steps, warm):
    """civic_anchor_aggregate (Eq. 8) on workload `w`: (result dict, tensors for further checks)."""
    import torch

    from paper_2605_28115_b200 import civic
    from paper_2605_28115_b200 import workloads as W

    x0, anchors = W.agg_inputs(w, dev)
    z0 = torch.empty((w.n_img, w.m_e, w.d_v), dtype=torch.bfloat16, device=dev)
    mass = torch.empty((w.n_img, w.t_e), dtype=torch.float32, device=dev)
    ws = torch.empty(civic.anchor_aggregate_workspace_bytes(w.n_img, w.t_e, w.m_e, w.d_v), dtype=torch.uint8, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)

    # The anchors are a learned constant at inference: Q_A is prepared once, outside the timed loop.
    # The call that prepares them every time is timed beside it (a shorter loop).
    prepared = civic.civic_anchor_prepare(anchors)

    def step():
        civic.civic_anchor_aggregate(x0, prepared, w.tau, z0=z0, token_mass=mass, workspace=ws, device_status=status)

    def step_unprepared():
        civic.civic_anchor_aggregate(x0, anchors, w.tau, z0=z0, token_mass=mass, workspace=ws, device_status=status)

    for _ in range(warm):
        step()
    torch.cuda.synchronize()
    sampler = ClockSampler(torch.device(dev).index or 0)
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    launches0 = civic.launch_count()
    sampler.start()
    start.record()
    for _ in range(steps):
        step()
    end.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    launches = civic.launch_count() - launches0
    ms = start.elapsed_time(end) / steps
    unprepared_us = time_loop(step_unprepared, steps, warm)  # as long a loop: the same power-cap regime
    if int(status.item()) != 0:
        raise SystemExit(f"a wait inside the aggregation kernels timed out (status {int(status.item())})")
    value = w.flops / (ms * 1e-3) / 1e12
    burst, sustained, which = measured_tensor_peak()
    timed_s = ms * 1e-3 * steps
    peak = sustained if timed_s > 0.5 else burst  # a long loop runs under the power cap
    roofline = {"bound": "tensor", "kernel": "civic_anchor_aggregate_prepared: four launches, of which the two tcgen05 "
                "contractions carry all the flops (the other two are memory-bound helpers and are inside the time)",
                "achieved": value, "peak": peak, "unit": "TFLOP/s", "frac": value / peak, "peak_source": which,
                "peak_kind": "sustained" if timed_s > 0.5 else "burst", "frac_of_burst_peak": value / burst,
                "traffic": None, "algorithmic_flops_per_step": w.flops, "us_per_step": ms * 1e3}
    res = {"workload": w.name, "steps": steps, "us_per_step": ms * 1e3, "value": value, "unit": "TFLOP/s",
           "constants": "anchors prepared once (civic_anchor_prepare), outside the timed loop",
           "us_per_step_preparing_the_anchors_every_call": unprepared_us,
           "gpu_launches": launches, "clocks": clocks, "roofline": roofline}
    return res, (x0, anchors, z0, mass, step)


def kv_attention_within_bound(q, k, v, r, n_heads, out):
    """Image 0 of a civic_kv_compressed_attention result against the fp64 oracle: the largest error as
    a share of the element-wise bound derived from the arithmetic, and the oracle's time."""
    import numpy as np

    from oracle import aggregate as OA

    q64, k64, v64 = (a[0].double().cpu().numpy() for a in (q, k, v))
    r64 = r.double().cpu().numpy()
    d = q64.shape[1] // n_heads
    t0 = time.perf_counter()
    want, k_c, v_c = OA.kv_compressed_attention(q64, k64, v64, r64, n_heads)
    seconds = time.perf_counter() - t0
    rbar = OA.column_normalize(r64)
    abs_kc, abs_vc = rbar.T @ np.abs(k64), rbar.T @ np.abs(v64)
    got = out[0].float().cpu().numpy().astype(np.float64)
    share = 0.0
    for h in range(n_heads):
        c = slice(h * d, (h + 1) * d)
        lam = 2.0 ** -8 * np.max(np.abs(q64[:, c]) @ abs_kc[:, c].T) / np.sqrt(d)
        eps_w = np.expm1(2 * lam) + 2.0 ** -8 * (1 + 2.0 ** -7)
        logits = q64[:, c] @ k_c[:, c].T / np.sqrt(d)
        wgt = np.exp(logits - logits.max(axis=1, keepdims=True))
        wgt /= wgt.sum(axis=1, keepdims=True)
        bound = (eps_w + 2.0 ** -8) * (wgt @ abs_vc[:, c]) + 2.0 ** -9 * np.abs(want[:, c])
        share = max(share, float(np.max(np.abs(got[:, c] - want[:, c]) / np.maximum(bound, 1e-300))))
    return share, float(np.max(np.abs(got - want))), seconds


def time_kv_attention(w, dev, steps, warm):
    """civic_kv_compressed_attention (Eq. 9) on workload `w`: (result dict, tensors for further checks)."""
    import torch

    from paper_2605_28115_b200 import civic
    from paper_2605_28115_b200 import workloads as W

    q, k, v, r = W.kvattn_inputs(w, dev)
    out = torch.empty_like(q)
    ws = torch.empty(civic.kv_compressed_attention_workspace_bytes(w.n_img, w.m_e, w.n_heads, w.head_dim, w.s),
                     dtype=torch.uint8, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)

    # R is a learned constant at inference: converted once, outside the timed loop.  The call that
    # converts it every time is timed beside it.
    prepared = civic.civic_kv_attention_prepare(r)

    def step():
        civic.civic_kv_compressed_attention(q, k, v, prepared, w.n_heads, out=out, workspace=ws, device_status=status)

    def step_unprepared():
        civic.civic_kv_compressed_attention(q, k, v, r, w.n_heads, out=out, workspace=ws, device_status=status)

    for _ in range(warm):
        step()
    torch.cuda.synchronize()
    sampler = ClockSampler(torch.device(dev).index or 0)
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    launches0 = civic.launch_count()
    sampler.start()
    start.record()
    for _ in range(steps):
        step()
    end.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    launches = civic.launch_count() - launches0
    ms = start.elapsed_time(end) / steps
    unprepared_us = time_loop(step_unprepared, steps, warm)
    if int(status.item()) != 0:
        raise SystemExit(f"a wait inside the kernels timed out (status {int(status.item())})")
    value = w.flops / (ms * 1e-3) / 1e12
    burst, _, which = measured_tensor_peak()
    roofline = {"bound": "tensor", "kernel": "civic_kv_compressed_attention_prepared (two launches; latency-bound at this size)",
                "achieved": value, "peak": burst, "unit": "TFLOP/s", "frac": value / burst, "peak_source": which,
                "peak_kind": "burst", "traffic": None, "algorithmic_flops_per_step": w.flops, "us_per_step": ms * 1e3}
    res = {"workload": w.name, "steps": steps, "us_per_step": ms * 1e3, "value": value, "unit": "TFLOP/s",
           "constants": "R prepared once (civic_kv_attention_prepare), outside the timed loop",
           "us_per_step_converting_r_every_call": unprepared_us,
           "gpu_launches": launches, "clocks": clocks, "roofline": roofline}
    return res, (q, k, v, r, out)


def other_workloads(dev, with_oracle):
    """What the default run measures after its main workload, each with its own clocks and its own
    comparison against the CPU oracle: the other K/V configurations (roofline fraction of the K/V
    launch), the small configurations (latency, plain and as a graph), Eq. 8 and Eq. 9."""
    import gc

    import torch

    from paper_2605_28115_b200 import workloads as W

    out = {}
    for wl, steps in ((W.C5_HALF, 200), (W.C5_THIRD, 200), (W.C5_QUARTER, 200),
                      (W.C1, 2000), (W.C2, 2000), (W.C4, 2000)):
        out[wl.name] = time_other_path_workload(wl, dev, steps, with_oracle)
        gc.collect()
        torch.cuda.empty_cache()
    w = W.AGG_896
    res, (x0, anchors, z0, mass, _) = time_aggregate(w, dev, 3000, 20)
    if with_oracle:
        share, err, _ = aggregate_within_bound(x0, anchors, w.tau, z0, mass)
        res.update(equals_oracle=share <= 1.0, largest_error_as_share_of_bound=share, largest_abs_error=err,
                   oracle_sample="image 0 of the batch, element-wise bound derived from the bf16 arithmetic")
    out[w.name] = res
    del x0, anchors, z0, mass
    w = W.KVATTN_896
    res, (q, k, v, r, o) = time_kv_attention(w, dev, 3000, 20)
    if with_oracle:
        share, err, _ = kv_attention_within_bound(q, k, v, r, w.n_heads, o)
        res.update(equals_oracle=share <= 1.0, largest_error_as_share_of_bound=share, largest_abs_error=err,
                   oracle_sample="image 0 of the batch, element-wise bound derived from the bf16 arithmetic")
    out[w.name] = res
    return out


def run_civic(args):
    import torch
    import torch.distributed as dist

    from paper_2605_28115_b200 import build as civic_build
    from paper_2605_28115_b200 import civic, sharding
    from paper_2605_28115_b200 import workloads as W

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if world != args.gpus:
        raise SystemExit(f"--gpus {args.gpus} but WORLD_SIZE={world}: launch with torch.distributed.run")
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU implementation")
    torch.cuda.set_device(local_rank)
    dev = f"cuda:{local_rank}"
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(dev))
    if rank == 0:
        civic_build.build()
    if world > 1:
        dist.barrier()
    civic.load()

    wl = pick_workload(args)
    st = DeviceState(wl, dev, rank, args.kv_layout, args.merge)
    nbytes = step_bytes(wl, st.merge)
    merge_on = st.merge
    default_variant = args.kv_layout == "token_major" and not merge_on

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    warm = max(args.warmup, 3)
    for _ in range(warm):
        st.step()
    barrier()

    # The K/V kernel is bracketed by events on every KV_EVENT_STRIDE-th timed step only: an event
    # record between two kernels takes away their programmatic launch overlap, so bracketing
    # every step would slow the very steps being timed.
    stride = max(1, min(KV_EVENT_STRIDE, args.steps // 20))
    kv_ev = {i: (torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
             for i in range(0, args.steps, stride)} if wl.n_layers else None
    graph, launches_per_replay = None, 0
    if args.graph:
        side = torch.cuda.Stream()
        with torch.cuda.stream(side):
            st.step()
            torch.cuda.synchronize()
            before_capture = civic.launch_count()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=side):
                st.step()
            launches_per_replay = civic.launch_count() - before_capture
        for _ in range(3):
            graph.replay()
        kv_ev = None  # no events inside a graph: the roofline object needs the plain mode
    sampler = ClockSampler(local_rank)
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    launches0 = civic.launch_count()
    sampler.start()
    barrier()
    start.record()
    for i in range(args.steps):
        if graph is not None:
            graph.replay()
        else:
            st.step(kv_ev.get(i) if kv_ev else None)
    end.record()
    barrier()
    clocks = sampler.stop()
    launches = launches_per_replay * args.steps if graph is not None else civic.launch_count() - launches0
    ms_per_step = sharding.max_over_ranks(start.elapsed_time(end), dev) / args.steps
    value = sharding.job_throughput_gbs(nbytes["total"], world, ms_per_step)

    roofline = None
    if kv_ev:
        roofline = kv_roofline(wl, nbytes["kv"], [a.elapsed_time(b) for a, b in kv_ev.values()], args.kv_layout,
                               default_variant)
        if default_variant:
            own = contiguous_copy_rate(st)
            roofline["same_kernel_keeping_every_row_gbs"] = own
            roofline["frac_of_same_kernel_keeping_every_row"] = roofline["achieved"] / own
            roofline["with_index_check"] = index_check_cost(st)

    # end to end: pinned host inputs -> path -> pinned host results, every step
    e2e = None
    if not args.no_e2e and default_variant:
        n_e2e = max(1, args.e2e_steps)
        modes = {}
        for mode in ("zero_copy", "staged") + (("pipelined",) if wl.n_layers else ()):
            hs = HostState(st, mode)
            hs.step()
            barrier()
            ok = hs.matches_device_results()
            hs.step()
            barrier()
            s2, e2 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            s2.record()
            for _ in range(n_e2e):
                hs.step()
            e2.record()
            barrier()
            ms_e2e = sharding.max_over_ranks(s2.elapsed_time(e2), dev) / n_e2e
            modes[mode] = {"value": sharding.job_throughput_gbs(nbytes["total"], world, ms_e2e),
                           "ms_per_step": ms_e2e, "h2d_bytes_per_step": hs.h2d_bytes,
                           "d2h_bytes_per_step": hs.d2h_bytes, "results_match_device_path": ok}
            del hs
        best = min((m for m in modes if m != "staged"), key=lambda m: modes[m]["ms_per_step"])
        e2e = {"value": modes[best]["value"], "unit": UNIT,
               "h2d_bytes_per_step": modes[best]["h2d_bytes_per_step"],
               "d2h_bytes_per_step": modes[best]["d2h_bytes_per_step"],
               "ms_per_step": modes[best]["ms_per_step"], "steps": n_e2e, "mode": best,
               "zero_copy_how": "the C-ABI calls get pinned host pointers for hidden and K/V sources and results: "
                                "the kernels pull only the kept rows over PCIe and write the compacted rows straight "
                                "to host memory; scores and pos ids are copied in, indices copied out",
               "zero_copy": modes["zero_copy"], "pipelined": modes.get("pipelined"),
               "pipelined_how": "as zero-copy for the reads, but the K/V kernel writes into device buffers two layers "
                                "per launch and a second stream copies each finished chunk to pinned host memory "
                                "while the kernel reads the next",
               "staged": modes["staged"],
               "staged_how": "cudaMemcpyAsync of every input to the device, device-resident path, "
                             "cudaMemcpyAsync of every result back",
               "results_match_device_path": modes[best]["results_match_device_path"]}

    cpu = None
    with_oracle = rank == 0 and world == 1 and not args.no_cpu_baseline and default_variant
    if with_oracle:
        cpu = cpu_baseline(st)
        st.step()
        torch.cuda.synchronize()
        cpu["gpu_result_equals_oracle"] = path_equals_oracle(st)

    # the other configurations, Eq. 8 and Eq. 9: only beside the default single-GPU measurement
    others = None
    if (rank == 0 and world == 1 and default_variant and not args.no_others and graph is None
            and args.workload == "c3_kv_qwen3vl8b" and not args.layers):
        import gc

        del st
        gc.collect()
        torch.cuda.empty_cache()
        others = other_workloads(dev, with_oracle)

    if rank == 0:
        variant = {} if default_variant else {"workload": wl.name + (
            "" if args.kv_layout == "token_major" else "+" + args.kv_layout) + ("+merge" if merge_on else "")}
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": warm, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "u8", "data": "synthetic",
                "config": config_of(wl, {"parallelism": parallelism_of(world), **variant}),
                "variant": {"cuda_graph": graph is not None, "kv_layout": args.kv_layout, "merge": merge_on},
                "bytes_per_step": nbytes, "gpu_launches": launches, "clocks": clocks,
                "roofline": roofline, "e2e": e2e, "cpu_baseline": cpu, "other_workloads": others}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


# ----------------------------------------------------------------------------- aggregation (Eq. 8)

def run_aggregate(args):
    """`--workload agg_*`: one step = one civic_anchor_aggregate call (anchor preparation, token
    statistics, the two tensor-core contractions, token mass) on a batch of images."""
    import torch

    from paper_2605_28115_b200 import build as civic_build
    from paper_2605_28115_b200 import civic
    from paper_2605_28115_b200 import workloads as W

    if int(os.environ.get("WORLD_SIZE", "1")) != 1 or args.gpus != 1:
        raise SystemExit("the aggregation workload is benchmarked on one GPU")
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU implementation")
    dev = "cuda:0"
    civic_build.build()
    civic.load()
    w = W.AGG_BY_NAME[args.workload]
    warm = max(args.warmup, 3)
    res, (x0, anchors, z0, mass, step) = time_aggregate(w, dev, args.steps, warm)
    ms = res["us_per_step"] * 1e-3

    # end to end: pinned host tokens in, compact rows and token mass back out
    e2e = None
    if not args.no_e2e:
        x_h = torch.empty(x0.shape, dtype=x0.dtype, pin_memory=True).copy_(x0)
        z_h = torch.empty(z0.shape, dtype=z0.dtype, pin_memory=True)
        m_h = torch.empty(mass.shape, dtype=mass.dtype, pin_memory=True)

        def host_step():
            x0.copy_(x_h, non_blocking=True)
            step()
            z_h.copy_(z0, non_blocking=True)
            m_h.copy_(mass, non_blocking=True)

        host_step()
        torch.cuda.synchronize()
        n_e2e = max(1, args.e2e_steps)
        s2, e2 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s2.record()
        for _ in range(n_e2e):
            host_step()
        e2.record()
        torch.cuda.synchronize()
        ms2 = s2.elapsed_time(e2) / n_e2e
        e2e = {"value": w.flops / (ms2 * 1e-3) / 1e12, "unit": "TFLOP/s", "ms_per_step": ms2, "steps": n_e2e,
               "h2d_bytes_per_step": x_h.numel() * 2, "d2h_bytes_per_step": z_h.numel() * 2 + m_h.numel() * 4,
               "results_match_device_path": bool(torch.equal(z_h, z0.cpu()))}

    cpu = None
    if not args.no_cpu_baseline:
        share, err, seconds = aggregate_within_bound(x0, anchors, w.tau, z0, mass)
        cpu = {"value": w.flops / w.n_img / seconds / 1e12, "unit": "TFLOP/s", "cores": os.cpu_count(), "kind": "oracle",
               "sample": f"the fp64 numpy oracle on ONE of the {w.n_img} images, one run, {seconds * 1e3:.0f} ms per image",
               "max_abs_difference_to_gpu_result": err, "largest_error_as_share_of_bound": share,
               "gpu_result_equals_oracle": share <= 1.0}

    line = {"metric": "aggregation_TFLOPs_eq8", "value": res["value"], "unit": "TFLOP/s", "n_gpus": 1, "steps": args.steps,
            "warmup": warm, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": {"workload": w.name, "n_img": w.n_img, "t_e": w.t_e, "m_e": w.m_e, "d_v": w.d_v, "tau": w.tau,
                       "l2": "the tokens (75 MB) and the weights W_A (67 MB) together exceed L2; no flush",
                       "parallelism": "single"},
            "gpu_launches": res["gpu_launches"], "clocks": res["clocks"], "roofline": res["roofline"], "e2e": e2e,
            "cpu_baseline": cpu}
    print(json.dumps(line), flush=True)


def run_kv_attention(args):
    """`--workload kvattn_*`: one step = one civic_kv_compressed_attention call (Eq. 9)."""
    import torch

    from paper_2605_28115_b200 import build as civic_build
    from paper_2605_28115_b200 import civic
    from paper_2605_28115_b200 import workloads as W

    if int(os.environ.get("WORLD_SIZE", "1")) != 1 or args.gpus != 1:
        raise SystemExit("this workload is benchmarked on one GPU")
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU implementation")
    dev = "cuda:0"
    civic_build.build()
    civic.load()
    w = W.KVATTN_BY_NAME[args.workload]
    warm = max(args.warmup, 3)
    res, (q, k, v, r, out) = time_kv_attention(w, dev, args.steps, warm)
    cpu = None
    if not args.no_cpu_baseline:
        share, err, seconds = kv_attention_within_bound(q, k, v, r, w.n_heads, out)
        cpu = {"value": w.flops / w.n_img / seconds / 1e12, "unit": "TFLOP/s", "cores": os.cpu_count(), "kind": "oracle",
               "sample": f"the fp64 numpy oracle on ONE of the {w.n_img} images, one run, {seconds * 1e3:.0f} ms",
               "max_abs_difference_to_gpu_result": err, "largest_error_as_share_of_bound": share,
               "gpu_result_equals_oracle": share <= 1.0}
    line = {"metric": "kv_compressed_attention_TFLOPs_eq9", "value": res["value"], "unit": "TFLOP/s", "n_gpus": 1,
            "steps": args.steps, "warmup": warm, "ms_per_step": res["us_per_step"] * 1e-3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": w.name, "n_img": w.n_img, "m_e": w.m_e, "n_heads": w.n_heads, "head_dim": w.head_dim,
                       "s": w.s, "l2": "working set (50 MB) smaller than L2 and not flushed: a latency figure",
                       "parallelism": "single"},
            "gpu_launches": res["gpu_launches"], "clocks": res["clocks"], "roofline": res["roofline"], "e2e": None,
            "cpu_baseline": cpu}
    print(json.dumps(line), flush=True)


def run_long_select(args):
    """`--workload longsel_*`: one step = one civic_select_large call on segments beyond one thread
    block; timed with the library's own chunking (which may take the one-launch cluster path) and
    with an explicit chunk of the same size (always the five launches), as a plain loop and as
    replays of a CUDA graph of one call."""
    import numpy as np
    import torch

    from paper_2605_28115_b200 import build as civic_build
    from paper_2605_28115_b200 import civic
    from paper_2605_28115_b200 import workloads as W

    if int(os.environ.get("WORLD_SIZE", "1")) != 1 or args.gpus != 1:
        raise SystemExit("this workload is benchmarked on one GPU")
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU implementation")
    dev = "cuda:0"
    civic_build.build()
    civic.load()
    wl = W.LONG_BY_NAME[args.workload]
    scores_host = W.scores(wl)
    scores = torch.from_numpy(scores_host).to(dev)
    desc = civic.SelectDesc(wl.t, wl.h, wl.w, wl.region_h, wl.region_w, wl.floor_m, wl.k)
    out = torch.empty((wl.n_seg, wl.k), dtype=torch.int32, device=dev)
    row = min(wl.region_h, wl.h) * wl.w
    explicit = max(2048, min(16384, (wl.n_seg * wl.n + 147) // 148))
    explicit = max(row, explicit // row * row)  # the default's size, rounded to whole region rows
    warm = max(args.warmup, 3)

    def timed(chunk):
        ws = torch.empty(civic.select_workspace_bytes(desc, wl.n_seg, chunk), dtype=torch.uint8, device=dev)
        call = lambda: civic.civic_select_large(scores, desc, keep_idx=out, workspace=ws, chunk_tokens=chunk)
        before = civic.launch_count()
        call()
        per_call = civic.launch_count() - before
        for _ in range(warm):
            call()
        torch.cuda.synchronize()
        start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        start.record()
        for _ in range(args.steps):
            call()
        end.record()
        torch.cuda.synchronize()
        plain_us = start.elapsed_time(end) / args.steps * 1e3
        graph, side = torch.cuda.CUDAGraph(), torch.cuda.Stream()
        with torch.cuda.stream(side):
            with torch.cuda.graph(graph, stream=side):
                call()
        for _ in range(warm):
            graph.replay()
        torch.cuda.synchronize()
        start.record()
        for _ in range(args.steps):
            graph.replay()
        end.record()
        torch.cuda.synchronize()
        return {"launches_per_call": per_call, "plain_loop_us": plain_us,
                "graph_replay_us": start.elapsed_time(end) / args.steps * 1e3}

    sampler = ClockSampler(0)
    launches0 = civic.launch_count()
    sampler.start()
    own, five = timed(0), timed(explicit)
    clocks = sampler.stop()
    launches = civic.launch_count() - launches0
    cpu = None
    if not args.no_cpu_baseline:  # the oracle as it stands, timed on the host cores; its result is compared too
        import oracle

        threads = oracle.default.set_threads(0)
        times = []
        for _ in range(3):
            t0 = time.perf_counter()
            want = oracle.default.select(scores_host, wl.t, wl.h, wl.w, wl.region_h, wl.region_w, wl.floor_m, wl.k)
            times.append(time.perf_counter() - t0)
        med = statistics.median(times)
        cpu = {"value": wl.n_seg * wl.n / med / 1e6, "unit": "Mtokens/s", "cores": threads, "kind": "oracle",
               "sample": f"the whole batch, median of 3 runs, {med * 1e3:.1f} ms",
               "gpu_result_equals_oracle": bool(np.array_equal(out.cpu().numpy(), want))}
    us = own["graph_replay_us"]
    line = {"metric": "long_segment_selection_Mtokens_per_s", "value": wl.n_seg * wl.n / us, "unit": "Mtokens/s",
            "n_gpus": 1, "steps": args.steps, "warmup": warm, "ms_per_step": us * 1e-3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "u32", "data": "synthetic",
            "config": {"workload": wl.name, "n_seg": wl.n_seg, "grid_thw": [wl.t, wl.h, wl.w],
                       "region_hw": [wl.region_h, wl.region_w], "floor_per_region": wl.floor_m, "k": wl.k,
                       "scores": wl.score_kind, "l2": "scores fit in L2 and are not flushed: a latency figure",
                       "parallelism": "single"},
            "own_chunking": own, "five_launches": dict(five, chunk_tokens=explicit),
            "gpu_launches": launches, "clocks": clocks,
            "roofline": {"bound": "latency", "kernel": "civic_select_large", "achieved": us, "peak": None, "unit": "us",
                         "frac": None, "traffic": None},
            "e2e": None, "cpu_baseline": cpu}
    print(json.dumps(line), flush=True)


def run_aggregate_reference(args):
    """The fp64 numpy oracle of Eq. 8 on this machine's host cores; each step is ONE image of the
    workload (a bounded sample), at most 10 steps."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    from oracle import aggregate as OA
    from paper_2605_28115_b200 import workloads as W

    w = W.AGG_BY_NAME[args.workload]
    x0, anchors = W.agg_inputs(w.__class__(w.name, 1, w.t_e, w.m_e, w.d_v, w.tau, w.seed), "cpu")
    x64, a64 = x0[0].double().numpy(), anchors.double().numpy()
    steps, warm = min(args.steps, 10), min(max(args.warmup, 1), 3)
    for _ in range(warm):
        OA.anchor_aggregate(x64, a64, w.tau)
    t0 = time.perf_counter()
    for _ in range(steps):
        OA.anchor_aggregate(x64, a64, w.tau)
    ms = (time.perf_counter() - t0) * 1e3 / steps
    value = w.flops / w.n_img / (ms * 1e-3) / 1e12
    sample = f"each step = the fp64 numpy oracle on one of the {w.n_img} images of the workload"
    line = {"impl": "reference", "metric": "aggregation_TFLOPs_eq8", "value": value, "unit": "TFLOP/s",
            "n_gpus": args.gpus, "steps": steps, "warmup": warm, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": w.name, "n_img": w.n_img, "t_e": w.t_e, "m_e": w.m_e, "d_v": w.d_v, "tau": w.tau,
                       "sample": sample},
            "cpu_baseline": {"value": value, "unit": "TFLOP/s", "cores": os.cpu_count(), "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": value, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------- reference arm

def run_reference(args):
    """The CPU oracle on this machine's host cores, same metric and workload; at most 50 steps."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import numpy as np

    import oracle
    from paper_2605_28115_b200 import workloads as W

    wl = pick_workload(args)
    o = oracle.default
    threads = o.set_threads(0)
    n_layers = wl.n_layers
    sample = wl
    rng = np.random.default_rng(wl.seed)
    row = wl.kv_heads * wl.head_dim

    def payload(shape):  # opaque 16-bit patterns; values never influence the path
        return rng.integers(0, 1 << 16, size=shape, dtype=np.uint16)

    scores = W.scores(wl)
    pos = W.pos_ids(wl)
    hidden = payload((wl.n_seg, wl.n, wl.hidden_dim)) if wl.hidden_dim else None
    ks = [payload((wl.n_seg, wl.seq_len, row)) for _ in range(n_layers)]
    vs = [payload((wl.n_seg, wl.seq_len, row)) for _ in range(n_layers)]
    nbytes = step_bytes(sample)["total"]

    def step():
        keep = o.select(scores, wl.t, wl.h, wl.w, wl.region_h, wl.region_w, wl.floor_m, wl.k)
        o.compact(hidden, pos, keep)
        if n_layers:
            o.compact_kv(ks, vs, o.seq_indices(keep, wl.seq_len, wl.text_before, wl.n))

    steps = min(args.steps, 50)
    warm = min(max(args.warmup, 3), 5)
    for _ in range(warm):
        step()
    t0 = time.perf_counter()
    for _ in range(steps):
        step()
    ms = (time.perf_counter() - t0) * 1e3 / steps
    value = nbytes / (ms * 1e-3) / 1e9
    sample_txt = (f"each step = whole path on {wl.n_seg} segments with all {n_layers} "
                  f"K/V layers on the host")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": steps, "warmup": warm, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "u8", "data": "synthetic",
            "config": config_of(wl, {"parallelism": parallelism_of(args.gpus)}),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle",
                             "sample": sample_txt},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


if __name__ == "__main__":
    a = parse_args()
    if a.workload.startswith("longsel_"):
        if a.impl == "reference":
            raise SystemExit("the reference arm covers the select + compact + KV and the aggregation workloads")
        run_long_select(a)
    elif a.workload.startswith("kvattn_"):
        if a.impl == "reference":
            raise SystemExit("the reference arm covers the select + compact + KV and the aggregation workloads")
        run_kv_attention(a)
    elif a.workload.startswith("agg_"):
        if a.impl == "reference":
            run_aggregate_reference(a)
        else:
            run_aggregate(a)
    elif a.impl == "reference":
        run_reference(a)
    else:
        run_civic(a)
