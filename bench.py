#!/usr/bin/env python
"""Benchmark of the OasisKV decode hot path on B200: one JSON line per run.

A "step" is one decode step of a workload: per layer, the KV append of the step's tokens into the
GPU-resident local window (the committed token written through to the CPU pool), sparse attention over
the working set staged by the previous step fused with block scoring by the draft queries, summary
update, top-k, delta selection with capped eviction, and the gather of the admitted blocks from the
full-KV pool in PINNED HOST MEMORY on side streams.  metric = tokens/s per layer = batch / (step time / layers).

  value            : queries resident in HBM, full KV in pinned host memory (the gather crosses the host link).
  e2e              : the same, plus every layer's queries copied host->device and outputs device->host inside
                     every step.
  value_hbm_mirror : the full KV mirrored in HBM (no host link): the compute-only step, for the exposed
                     transfer time  value.ms_per_step - value_hbm_mirror.ms_per_step.
Consecutive steps are captured into CUDA graphs of `--group` steps; inside a graph a layer's transfer only
has to land before that layer's next-step attention (Sec. 4.2.2), so steps overlap.  The graphs of the timed
steps are instantiated and uploaded to the device before the timed region (the first replay of a graph of some
thousand nodes otherwise spends about 3 ms on the host before the device sees its first node).  After the timed
region the same K steps are replayed `--again` more times (default 2), each replay timed by itself and reported as
`ms_per_step_again` beside `value` and `e2e` (never part of them): the host link of a shared machine does not always
deliver the same rate, and a reader should see whether the timed region repeats.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--config 0..4] [--fetch-ratio R] [--group G]
                  [--repeats R] [--sweep-ratios 0.01,0.02,...] [--summary FILE] [--impl reference]

--config picks the workload (default 1, the reasoning-style decode the metric is quoted on; 0 and 4 rotate
over independent copies of their single layer so that every launch reads cold data; 4 prints one line with
a cell per budget x draft length).  --sweep-ratios repeats value / value_hbm_mirror / e2e for several fetch
caps (Sec. 5.5.1) and reports the exposed time per layer; --summary writes the numbers as a markdown table.
"""
import argparse
import json
import math
import os
import re
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

from paper_2608_08097_b200 import synth  # noqa: E402

METRIC = "sparse decode-attn+select tokens/s per layer"
UNIT = "tokens/s/layer"
BUDGETS = (32, 64, 128, 256, 512)        # configs[4]: K blocks = 512 .. 8,192 tokens
DRAFTS = (1, 2, 4, 8)


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=1, choices=[0, 1, 2, 3, 4])
    ap.add_argument("--layers", type=int, default=None, help="override the number of layers (debugging, profiling)")
    ap.add_argument("--batch", type=int, default=None, help="override the batch (debugging)")
    ap.add_argument("--context", type=int, default=None, help="override the context length (debugging)")
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--fetch-ratio", type=float, default=0.05, help="cap of the delta gather, fraction of K")
    ap.add_argument("--group", type=int, default=0, help="decode steps per CUDA graph (0: all timed steps in one)")
    ap.add_argument("--wait-group", type=int, default=0,
                    help="layers per pick-up of the side streams' events (0: a quarter of the layers, at most 8)")
    ap.add_argument("--transfer-group", type=int, default=0,
                    help="layers per gather launch when the pool is in host memory (0: up to 8 when the host link bounds the step, else 2)")
    ap.add_argument("--transfer-kind", default="", choices=["", "warp", "bulk"],
                    help="gather from host memory: warp per entry, or bulk copies through shared memory (default: bulk where "
                         "the host link bounds the step)")
    ap.add_argument("--repeats", type=int, default=1, help="replay the timed steps this many times in a second, long "
                                                            "timed region (reported as `sustained`)")
    ap.add_argument("--again", type=int, default=2, help="further replays of the timed steps, each timed by itself and "
                                                         "reported as ms_per_step_again (not part of value)")
    ap.add_argument("--sweep-ratios", default="", help="comma-separated fetch ratios to sweep (e.g. 0.01,0.02,0.05)")
    ap.add_argument("--summary", default="", help="write a markdown summary of the numbers to this file")
    ap.add_argument("--skip-e2e", action="store_true")
    ap.add_argument("--skip-cpu", action="store_true")
    ap.add_argument("--skip-mirror", action="store_true")
    return ap.parse_args()


def workload(args):
    """(configuration, description).  configs[0] and configs[4] have one layer: they run as 32 / 4 independent
    copies of it (different seeds), so that consecutive launches read different data."""
    base = (synth.C1, synth.C2, synth.C3, synth.C4, synth.C5)[args.config]
    kw = {}
    if args.config == 0:
        kw["layers"] = 32
    if args.config == 4:
        kw.update(layers=4, n_draft=max(DRAFTS))
    if args.layers:
        kw["layers"] = args.layers
    if args.batch:
        kw["batch"] = args.batch
    if args.context:
        kw["context"] = args.context
    kw["steps"] = max(base.steps, args.steps + max(args.warmup, 3) + 1)
    cfg = synth.scaled(base, **kw)
    names = ("configs[0] single layer, batch 1 (run as %d independent copies)" % cfg.layers,
             "configs[1] reasoning-style decode", "configs[2] long-context large batch",
             "configs[3] larger-model GQA-8 shape",
             "configs[4] budget x draft-length sweep (one layer run as %d independent copies)" % cfg.layers)
    return cfg, names[args.config]


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def profile_traffic(name="c2_layer_tcgen05_kernel.md"):
    """DRAM bytes (read + write) per launch of the fused kernel from the tracked ncu summary of the configs[1]
    shapes: the mean of the 'traffic (read + write)' row."""
    try:
        with open(os.path.join(ROOT, "profiles", name)) as f:
            for line in f:
                if line.startswith("| traffic (read + write)"):
                    vals = [float(x) for x in re.findall(r"([0-9.]+) MB", line)]
                    if vals:
                        return sum(vals) / len(vals) * 1e6
    except OSError:
        pass
    return None


def pick_transfer_group(link_ratio, layers, compute_us):
    """Layers per gather launch for a step whose layers spend `link_ratio` times as long on the host link as on scoring +
    attention (`compute_us` per layer); the measurements behind the thresholds are listed in Bench.transfer_group."""
    if link_ratio > 2.0 and layers >= 8:
        return min(8, layers // 2)
    if link_ratio > 1.0:
        return max(1, min(8, layers // 4))
    # near the break-even two layers per launch, unless a layer is so short that waiting for the second one's plan
    # costs more than the launch saves
    return max(1, min(2, layers // 4)) if link_ratio > 0.5 and compute_us >= 30.0 else 1


class ClockSampler:
    """Samples the SM clock and the clock-event (throttle) reasons through NVML, read-only,
    every few milliseconds from a thread while a timed region runs."""
    REASONS = (("hw_slowdown", 0x8), ("hw_thermal_slowdown", 0x40), ("sw_thermal_slowdown", 0x20),
               ("sw_power_cap", 0x4))

    def __init__(self, index):
        self.index, self.thread, self.stop_flag = index, None, threading.Event()
        self.clocks, self.reason_bits, self.max_mhz = [], 0, None

    def _open(self):
        """NVML set-up, done before the timed region starts (the first nvmlInit of a process can take longer than a
        short timed region)."""
        try:
            import pynvml
            pynvml.nvmlInit()
            visible = os.environ.get("CUDA_VISIBLE_DEVICES")
            idx = self.index
            if visible:
                try:
                    idx = int(visible.split(",")[self.index])
                except ValueError:
                    pass
            self._nvml = pynvml
            self._handle = pynvml.nvmlDeviceGetHandleByIndex(idx)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self._handle, pynvml.NVML_CLOCK_SM)
        except Exception:          # NVML missing or refused: report no samples
            self._nvml = self._handle = None

    def _run(self):
        try:
            nv, h = self._nvml, self._handle
            while not self.stop_flag.is_set():
                self.clocks.append(nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM))
                self.reason_bits |= int(nv.nvmlDeviceGetCurrentClocksEventReasons(h))
                time.sleep(0.002)
        except Exception:
            pass

    def start(self):
        self._open()
        if self._handle is None:
            return
        self.thread = threading.Thread(target=self._run, daemon=True)
        self.thread.start()

    def stop(self):
        self.stop_flag.set()
        if self.thread is not None:
            self.thread.join(timeout=2)
        out = {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": len(self.clocks)}
        if self.clocks:
            c = sorted(self.clocks)
            out["sm_mhz"] = c[len(c) // 2]
            out["reasons"] = [n for n, bit in self.REASONS if self.reason_bits & bit]
        return out


def dist_setup(args):
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl" if torch.cuda.is_available() else "gloo")
    return world, rank, local


def barrier(world):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()


def max_over_ranks(x, world, device):
    if world == 1:
        return x
    import torch.distributed as dist
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def time_pinned_h2d(device):
    """Pinned host -> device copy bandwidth, 1 GiB, best of 10 (GB/s)."""
    n = 1 << 30
    src = torch.empty(n, dtype=torch.uint8, pin_memory=True)
    dst = torch.empty(n, dtype=torch.uint8, device=device)
    best = 0.0
    for _ in range(10):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        dst.copy_(src, non_blocking=True)
        b.record()
        b.synchronize()
        best = max(best, n / (a.elapsed_time(b) * 1e-3) / 1e9)
    del src, dst
    return best


# ------------------------------------------------------------------------------------------- ours


class Work:
    """One (budget, draft length) view of the generated workload: contiguous per-layer query / new-KV tensors."""

    def __init__(self, bench, k, td):
        cfg = bench.cfg
        self.k, self.td, self.T = k, td, td + 1
        full = td == cfg.n_draft
        self.q_dev = [q if full else q[:, :, :self.T].contiguous() for q in bench.q_dev]              # [S][B][T][Hq][d]
        self.q_true_dev = [q if full else q[:, :, :td].contiguous() for q in bench.q_true_dev]        # [S][B][Td][Hq][d]
        self.new_kv = [t if full else t[:, :, :self.T].contiguous() for t in bench.new_kv]            # [S][B][T][Hkv][2][d]
        self.q_pinned = None

    def e2e_buffers(self, bench):
        """Pinned queries of every step stacked over the layers ([S][n_layers][B][T][Hq][128]), one device staging
        tensor and one pinned output tensor of the same per-step shape."""
        cfg = bench.cfg
        if self.q_pinned is None:
            self.q_pinned = torch.stack([q.cpu() for q in self.q_dev], dim=1).pin_memory()
            self.q_stage = torch.empty_like(self.q_pinned[0], device=bench.dev)
            self.out_pinned = torch.empty((cfg.layers, cfg.batch, self.T, cfg.n_q_heads, 128), dtype=torch.bfloat16,
                                          pin_memory=True)
        return self.q_pinned, self.q_stage, self.out_pinned


class Bench:
    def __init__(self, args, cfg, device, rank):
        from paper_2608_08097_b200 import build
        build.build()
        from paper_2608_08097_b200 import binding, pipeline
        binding.lib()
        self.args, self.cfg, self.dev, self.rank = args, cfg, device, rank
        self.binding, self.pipeline = binding, pipeline
        self.n_layers = cfg.layers
        self.host_kv, self.mirror, self.tables = [], [], []
        self.q_dev, self.q_true_dev, self.new_kv = [], [], []
        self.sample_layer = None
        self.err_word = torch.zeros(1, dtype=torch.int32, device=device)
        binding.set_error_word(self.err_word)

    def check_error_word(self, where):
        code = int(self.err_word.item())
        if code != 0:
            raise RuntimeError("a kernel's bounded wait ran out (code %d) during %s: the numbers are void" % (code, where))

    def generate(self, want_mirror, want_host):
        cfg = self.cfg
        t0 = time.time()
        for l in range(self.n_layers):
            P = cfg.batch * cfg.max_blocks
            host = torch.empty((P, cfg.n_kv_heads, 2, 16, 128), dtype=torch.bfloat16, pin_memory=True)
            lay = synth.make_layer(cfg, seed=self.args.seed + 7919 * self.rank, layer=l, device=self.dev, out_kv=host)
            self.tables.append(lay.block_table.to(self.dev))
            self.q_dev.append(lay.q_steps.to(self.dev))
            self.q_true_dev.append(lay.q_true_steps.to(self.dev))
            self.new_kv.append(synth.new_kv_steps(lay).to(self.dev))
            if want_mirror:
                self.mirror.append(host.to(self.dev, non_blocking=False))
            if want_host:
                self.host_kv.append(host)
            if l == 0:
                self.seq_steps = lay.seq_len_steps.clone()
                self.sample_layer = lay if want_host else None
            if not want_host:
                del host
        seq = self.seq_steps                                            # [S][B] int32 (host)
        self.seq_dev = seq.to(self.dev)
        self.first_dev = (seq // 16).to(torch.int32).to(self.dev)       # full blocks before the step's commit
        self.seq_next_dev = (seq + 1).to(torch.int32).to(self.dev)
        self.nfull_next_dev = ((seq + 1) // 16).to(torch.int32).to(self.dev)
        self.n_new_dev = (self.nfull_next_dev - self.first_dev).contiguous()
        self.gen_seconds = time.time() - t0

    def transfer_group(self, w, cap):
        """Layers per gather launch from pinned host memory, from the ratio of a layer's gather time on the link to its
        scoring + attention time.  Measured (step in ms, bulk gather unless noted): configs[1] (32 layers, ratio 3): 4.01
        with 8 layers per launch (16: the same; all 32: 5.37), 4.03 with 4, 4.11 with 2; configs[3] (8 layers, ratio 2.4): 1.11 with 4, 1.25 with 2,
        1.27 with 1; configs[2] (4 layers, ratio 1.3): 1.11 with 1, 1.17 with 2, 2.05 with 4 (the whole step's transfers
        then wait for its last layer); configs[1] at fetch ratio 0.02 (ratio 0.85, warp gather): 1.67 with 2, 1.75
        with 1 or 4; far below the break-even one launch per layer is best (configs[0]: 0.55-0.60 against 0.67-0.69 end
        to end)."""
        if self.args.transfer_group > 0:
            return self.args.transfer_group
        return pick_transfer_group(self.link_ratio(w, cap), self.cfg.layers, self.compute_us(w))

    def link_ratio(self, w, cap):
        """A layer's gathered bytes at 0.9 of the pinned copy peak over its scoring + attention bytes at 0.85 of the HBM
        copy peak: above 1 the host link bounds the step."""
        cfg = self.cfg
        link_us = cap * cfg.batch * cfg.n_kv_heads * 8192 / (0.9 * self.h2d_peak * 1e3)
        return link_us / self.compute_us(w)

    def compute_us(self, w):
        """A layer's scoring + attention bytes at 0.85 of the HBM copy peak, at least the 10 us a fused launch takes."""
        score, attn = algorithmic_bytes(self.cfg, w.k, w.T, self.seq_steps, [0])
        return max(10.0, (score + attn) / (0.85 * self.hbm_peak * 1e3))

    def link_bound(self, w, cap):
        return self.link_ratio(w, cap) > 1.0

    def wait_group(self):
        """Layers whose side-stream events the foreground stream picks up together: few enough that a step's last
        transfers overlap the next step's first layers, many enough to keep most consecutive fused launches
        overlapping."""
        return self.args.wait_group if self.args.wait_group > 0 else max(1, min(8, self.cfg.layers // 4))

    def engine(self, w, kv_list, cap):
        cfg = self.cfg
        # gathers from pinned host memory alternate between three transfer streams (a gather's first requests are in
        # flight while the previous gather's last ones come back)
        host_pool = len(kv_list) > 0 and not kv_list[0].is_cuda
        eng = self.pipeline.DecodeEngine(cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.max_blocks, w.k, w.T,
                                         self.n_layers, self.dev, mode="delta", cap=cap, append=True,
                                         transfer_streams=getattr(self.args, "transfer_streams", 1),
                                         plan_stream=getattr(self.args, "plan_stream", "own"), wait_group=self.wait_group(),
                                         n_commit=getattr(self.args, "n_commit", 1),
                                         # (pool in pinned host memory: bulk gather where the link bounds the step, else a
                                         #  small warp gather -- 32 thread blocks -- that disturbs the fused kernel least)
                                         transfer_kind=(getattr(self.args, "transfer_kind", "") or
                                                        ("bulk" if host_pool and self.link_bound(w, cap) else "warp")),
                                         transfer_ctas=(getattr(self.args, "transfer_ctas", 0) or
                                                        (32 if host_pool and not self.link_bound(w, cap) else 0)),
                                         transfer_group=self.transfer_group(w, cap) if host_pool else 1)
        for l in range(self.n_layers):
            eng.attach(l, kv_list[l], self.tables[l])
        eng.prime([w.q_dev[l][0] for l in range(self.n_layers)], self.first_dev[0].contiguous(), self.seq_dev[0].contiguous())
        return eng

    def step_args(self, w, s, e2e):
        n = self.n_layers
        kw = dict(step_stamp=s + 1, new_kv=[w.new_kv[l][s] for l in range(n)])
        if e2e:
            q_pinned, q_stage, out_pinned = w.e2e_buffers(self)
            q_list = q_stage
            kw.update(q_host=q_pinned[s], out_host=out_pinned)
        else:
            q_list = [w.q_dev[l][s] for l in range(n)]
        args = (q_list, self.seq_dev[s], self.first_dev[s], self.n_new_dev[s], self.nfull_next_dev[s],
                self.seq_next_dev[s])
        return args, kw

    def timed(self, eng, w, world, W, K, e2e=False, repeats=1):
        """The steps are captured into CUDA graphs of `--group` consecutive steps (default: all K timed steps in
        one); W warm-up steps are replayed, then exactly K timed steps bracketed by barrier + synchronize.
        Returns (ms per step, clocks, launches, sustained) -- `sustained`: the K steps replayed `repeats` times."""
        group = self.args.group if self.args.group > 0 else K
        warm = eng.capture_steps([self.step_args(w, s, e2e) for s in range(W)])
        graphs = [eng.capture_steps([self.step_args(w, s, e2e) for s in range(s0, min(s0 + group, W + K))])
                  for s0 in range(W, W + K, group)]
        eng.replay(warm)
        for g in graphs:                # instantiated and uploaded ahead of the timed region, like any other set-up
            eng.upload(g)
        torch.cuda.synchronize()
        sampler = ClockSampler(self.dev.index or 0)
        sampler.start()
        barrier(world)
        torch.cuda.synchronize()
        start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        l0 = eng.launches
        start.record(eng.main)
        for g in graphs:
            eng.replay(g)
        end.record(eng.main)
        torch.cuda.synchronize()
        barrier(world)
        clocks = sampler.stop()
        launches = eng.launches - l0
        ms = max_over_ranks(start.elapsed_time(end) / K, world, self.dev)
        self.check_error_word("the timed steps")
        # the same K steps twice more, each replay timed by itself: not part of `value`, reported beside it so that a
        # reader sees how far one timed region on this (shared) machine repeats
        self.again_ms = []
        for _ in range(max(0, self.args.again)):
            torch.cuda.synchronize()
            start.record(eng.main)
            for g in graphs:
                eng.replay(g)
            end.record(eng.main)
            torch.cuda.synchronize()
            self.again_ms.append(round(max_over_ranks(start.elapsed_time(end) / K, world, self.dev), 4))
        sustained = None
        if repeats > 1:
            # a long timed region: the same K steps again and again (the working sets keep evolving; the shapes and
            # the per-step traffic stay what they are), with the clocks sampled throughout
            sampler = ClockSampler(self.dev.index or 0)
            sampler.start()
            torch.cuda.synchronize()
            start.record(eng.main)
            for _ in range(repeats):
                for g in graphs:
                    eng.replay(g)
            end.record(eng.main)
            torch.cuda.synchronize()
            c = sampler.stop()
            ms_r = max_over_ranks(start.elapsed_time(end) / (K * repeats), world, self.dev)
            sustained = {"ms_per_step": round(ms_r, 4), "seconds": round(ms_r * K * repeats * 1e-3, 2), "repeats": repeats,
                         "sm_mhz_median": c["sm_mhz"], "reasons": c["reasons"],
                         "ms_x_mhz": None if c["sm_mhz"] is None else round(ms_r * c["sm_mhz"], 1)}
            self.check_error_word("the repeated steps")
        return ms, clocks, launches, sustained

    def kernel_solo_times(self, eng, w, s):
        """Launch durations (us) of the scoring, the attention and the fused kernel on their own.
        graph: one launch per layer (all layers' distinct buffers, far more than L2) captured into a CUDA graph on
        one stream and replayed, timed with CUDA events on that stream -- consecutive fused launches overlap there
        through programmatic dependent launch, as they do in the step.
        single: one launch alone with cold caches: a graph of [write 512 MB, the launch] minus a graph of [write
        512 MB] (the write flushes L2, keeps the neighbours apart, and its own time and the host's launch latency
        cancel in the difference); the median over up to four layers."""
        out, single = {}, {}
        st = eng.main
        flush = torch.empty(512 << 20, dtype=torch.uint8, device=self.dev)
        calls = {
            "score": lambda l: eng.layers[l].score(w.q_dev[l][s], self.nfull_next_dev[s]),
            "attn": lambda l: eng.layers[l].attend(w.q_dev[l][s], self.seq_dev[s], blk_tbl=eng.blk_tbl(l)),
        }
        if eng.fused:        # the launch the step actually makes: attention + scoring of a layer in one kernel
            calls["layer"] = lambda l: eng.layers[l].attend_and_score(w.q_dev[l][s], self.seq_dev[s], self.nfull_next_dev[s],
                                                                      blk_tbl=eng.blk_tbl(l))

        def graph_of(fn):
            torch.cuda.synchronize()
            with torch.cuda.stream(st):
                fn()
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=st, capture_error_mode="thread_local"):
                fn()
            return g

        def best_of(g, reps=5):
            best = None
            for _ in range(reps):
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                with torch.cuda.stream(st):
                    a.record(st)
                    g.replay()
                    b.record(st)
                torch.cuda.synchronize()
                t = a.elapsed_time(b) * 1e3
                best = t if best is None else min(best, t)
            return best

        t_flush = best_of(graph_of(lambda: flush.zero_()))
        for name, fn in calls.items():
            out[name] = best_of(graph_of(lambda: [fn(l) for l in range(self.n_layers)])) / self.n_layers
            ts = []
            for l in range(0, self.n_layers, max(1, self.n_layers // 4)):
                ts.append(best_of(graph_of(lambda: (flush.zero_(), fn(l)))) - t_flush)
            ts.sort()
            single[name] = ts[len(ts) // 2]
        del flush
        return out, single

    def recall(self, eng, w, steps):
        """Share of the draft-predicted top-k also chosen by the true next-step queries (same estimator)."""
        tot, n = 0.0, 0
        for l in range(0, self.n_layers, max(1, self.n_layers // 4)):
            L = eng.layers[l]
            sel_true = torch.empty_like(L.sel)
            for s in steps:
                with torch.cuda.stream(eng.main):
                    L.score(w.q_dev[l][s], self.nfull_next_dev[s])
                    L.select(self.nfull_next_dev[s], self.seq_next_dev[s], self.tables[l])
                    sel_draft = L.sel.clone()
                    L.score_queries(w.q_true_dev[l][s], self.nfull_next_dev[s])
                    L.select(self.nfull_next_dev[s], self.seq_next_dev[s], self.tables[l], sel=sel_true)
                eng.main.synchronize()
                a = sel_draft[..., :w.k]
                b = sel_true[..., :w.k]
                hit = (a[..., :, None] == b[..., None, :]).any(-1).float().mean().item()
                tot, n = tot + hit, n + 1
        return tot / max(n, 1)


def algorithmic_bytes(cfg, k, T, seq_steps, steps):
    """Per-launch algorithmic bytes of the scoring and attention kernels, averaged over steps."""
    B, Hkv, Hq = cfg.batch, cfg.n_kv_heads, cfg.n_q_heads
    score, attn = 0.0, 0.0
    for s in steps:
        L = seq_steps[s].to(torch.int64)
        nfull_next = (L + 1) // 16
        score += float((nfull_next * Hkv * (512 + 4)).sum())
        nfull = L // 16
        n_local = (L + T + 15) // 16 - nfull
        cols = torch.minimum(nfull, torch.tensor(k)) + n_local
        attn += float((cols * Hkv * 8192).sum()) + 2.0 * B * T * Hq * 128 * 2
    return score / len(steps), attn / len(steps)


def cpu_leg(bench, w, cfg, sel_gpu, s_sel, budget_s=12.0, mass_requests=2):
    """What runs on the host cores: (1) the oracle, as it stands, on one layer of one step, request by request
    (score + top-k + gather + attention), until about `budget_s` seconds are spent; (2) the secondary recall: the
    GPU's lookahead selection of step `s_sel` (layer 0) against the top-K blocks by the attention mass that the true
    next-step queries put on them, computed by the oracle's dense softmax for the first `mass_requests` requests."""
    import numpy as np
    from oracle import oracle
    oracle.lib()
    lay = bench.sample_layer
    kv = synth.u16(lay.host_kv)
    table = lay.block_table.numpy()
    scale = np.float32(1.0 / math.sqrt(128.0))
    done, t_used, steps_used = 0, 0.0, 0
    for s in range(min(lay.seq_len_steps.shape[0], 16)):           # step by step, request by request, until the budget is spent
        for b in range(cfg.batch):
            tb = table[b:b + 1]
            n_full = lay.n_full_steps[s].numpy()[b:b + 1]
            seq = lay.seq_len_steps[s].numpy()[b:b + 1]
            q = synth.u16(lay.q_steps[s][b:b + 1, :w.T].contiguous())
            summ = oracle.build_summaries(kv, tb, np.zeros(1, np.int32), n_full)          # set-up, not timed
            t0 = time.perf_counter()
            s32, _ = oracle.score_blocks(q[:, 1:], summ, n_full)
            sel, idx, slots = oracle.select_topk(s32, n_full, seq, w.T, w.k, tb)
            pool = np.zeros((cfg.n_kv_heads * (w.k + 2), 2, 16, 128), np.uint16)
            oracle.stage_blocks(kv.reshape(-1, 2, 16, 128), idx, slots, pool)
            oracle.sparse_attn(q, pool, slots.reshape(1, cfg.n_kv_heads, -1), sel, seq, scale, cfg.n_kv_heads)
            t_used += time.perf_counter() - t0
            done += 1
            if t_used >= budget_s:
                break
        steps_used = s + 1
        if t_used >= budget_s:
            break
    base = {"value": done / t_used, "unit": UNIT, "cores": 1, "host_cores": os.cpu_count(), "kind": "oracle",
            "sample": "layer 0, %d (request, step) units of steps 0..%d (batch %d), score+top-k+gather+attention each, single "
                      "thread (%.1f s)" % (done, steps_used - 1, cfg.batch, t_used)}
    # secondary recall (attention mass): the true queries of steps s+1.. sit at positions L_s + 1 + t
    recall_mass = None
    if sel_gpu is not None:
        nb = min(mass_requests, cfg.batch)
        seq_next = (lay.seq_len_steps[s_sel][:nb] + 1).numpy().astype(np.int32)
        q_true = synth.u16(lay.q_true_steps[s_sel][:nb, :w.td].contiguous())
        mass = oracle.block_mass(q_true, kv, table[:nb], seq_next, scale)
        n_full_next = (seq_next // 16).astype(np.int32)
        sel_mass = oracle.select_topk(mass.astype(np.float32), n_full_next, seq_next, w.T, w.k, table[:nb], want_stage=False)
        recall_mass = {"value": round(oracle.topk_recall(sel_gpu[:nb], sel_mass, w.k), 4),
                       "sample": "layer 0, step %d, requests 0..%d: GPU lookahead selection vs top-%d blocks by the true "
                                 "next-step queries' dense softmax mass (oracle, fp64)" % (s_sel, nb - 1, w.k)}
    return base, recall_mass


def kernel_rooflines(per_kernel, single, score_bytes, attn_bytes, hbm_peak):
    kern = {}
    for name, nbytes in (("score", score_bytes), ("attn", attn_bytes), ("layer", score_bytes + attn_bytes)):
        if name in per_kernel:
            gbs = nbytes / (per_kernel[name] * 1e-6) / 1e9
            kern[name] = {"us": round(per_kernel[name], 2), "algorithmic_MB": round(nbytes / 1e6, 2),
                          "GBps": round(gbs, 1), "frac_of_measured": round(gbs / hbm_peak, 3),
                          "frac_of_8TBps": round(gbs / 8000.0, 3)}
            if name in single:
                kern[name]["us_single_launch"] = round(single[name], 2)
                kern[name]["frac_single_launch"] = round(nbytes / (single[name] * 1e-6) / 1e9 / hbm_peak, 3)
    return kern


def admitted_entries(eng):
    """Gather requests actually issued by the last step, per layer."""
    return sum(int((p >= 0).sum().item()) for p in eng.plan_idx) / max(1, eng.n_layers)


def measure(bench, w, world, W, K, cap, hbm_peak, h2d_peak, want_mirror=True, want_host=True, want_e2e=True,
            want_kernels=True, repeats=1):
    """All timings of one (workload view, cap): the step with the pool mirrored in HBM, with the pool in pinned host
    memory, end to end; the kernels alone; recall."""
    cfg = bench.cfg
    n = cfg.layers
    steps = range(W, W + K)
    score_bytes, attn_bytes = algorithmic_bytes(cfg, w.k, w.T, bench.seq_steps, steps)
    tok = cfg.batch * world * n          # tokens/s/layer = batch / (step time / layers)
    qo_bytes = cfg.batch * w.T * cfg.n_q_heads * 128 * 2
    commit_bytes = cfg.batch * cfg.n_kv_heads * 512
    r = {"k_blocks": w.k, "n_draft": w.td, "cap": cap, "algorithmic_MB_per_layer": round((score_bytes + attn_bytes) / 1e6, 2)}
    sel_gpu = None
    if want_mirror and bench.mirror:
        eng = bench.engine(w, bench.mirror, cap)
        ms, clocks, launches, _ = bench.timed(eng, w, world, W, K)
        r["mirror"] = {"ms_per_step": round(ms, 4), "value": round(tok / (ms * 1e-3), 1), "launches": launches}
        gbs = (score_bytes + attn_bytes) * n / (ms * 1e-3) / 1e9
        r["step_hbm"] = {"achieved_GBps": round(gbs, 1), "frac_of_measured": round(gbs / hbm_peak, 3),
                         "note": "scoring + attention bytes of all layers / step time, full KV mirrored in HBM"}
        r["recall_lookahead_topk"] = round(bench.recall(eng, w, range(W, min(W + 4, W + K))), 4)
        if want_kernels:
            solo, single = bench.kernel_solo_times(eng, w, W)
            kern = kernel_rooflines(solo, single, score_bytes, attn_bytes, hbm_peak)
            r["kernels"] = kern
            r["dominant"] = "layer" if "layer" in solo else max(("score", "attn"), key=lambda x: solo.get(x, 0.0))
        bench.check_error_word("the HBM-mirror runs")
        del eng
        torch.cuda.empty_cache()
    if want_host and bench.host_kv:
        eng = bench.engine(w, bench.host_kv, cap)
        ms, clocks, launches, sustained = bench.timed(eng, w, world, W, K, repeats=repeats)
        n_req = admitted_entries(eng)
        gather = n * n_req * 8192
        r["host"] = {"ms_per_step": round(ms, 4), "value": round(tok / (ms * 1e-3), 1), "launches": launches,
                     "clocks": clocks, "requests_per_layer": round(n_req, 1),
                     "h2d_bytes_per_step": int(gather), "d2h_bytes_per_step": int(n * commit_bytes),
                     "gather_GBps_over_step": round(gather / (ms * 1e-3) / 1e9, 2),
                     "gather_frac_of_h2d_peak": round(gather / (ms * 1e-3) / 1e9 / h2d_peak, 3)}
        r["host"]["ms_per_step_again"] = list(bench.again_ms)
        if sustained:
            r["host"]["sustained"] = sustained
        if "mirror" in r:
            r["host"]["exposed_us_per_layer"] = round((ms - r["mirror"]["ms_per_step"]) * 1e3 / n, 2)
            r["host"]["compute_to_host_step_ratio"] = round(r["mirror"]["ms_per_step"] / ms, 3)
        # the GPU's lookahead selection of the last timed step, layer 0 (for the secondary recall on the host)
        sel_gpu = eng.layers[0].sel.cpu().numpy()
        r["_sel_step"] = W + K - 1
        del eng
        torch.cuda.empty_cache()
    if want_e2e and bench.host_kv:
        eng = bench.engine(w, bench.host_kv, cap)
        ms, clocks, launches, _ = bench.timed(eng, w, world, W, K, e2e=True)
        n_req = admitted_entries(eng)
        gather = n * n_req * 8192
        h2d = gather + n * qo_bytes
        r["e2e"] = {"value": round(tok / (ms * 1e-3), 1), "unit": UNIT, "h2d_bytes_per_step": int(h2d),
                    "d2h_bytes_per_step": int(n * (qo_bytes + commit_bytes)), "ms_per_step": round(ms, 4), "steps": K,
                    "ms_per_step_again": list(bench.again_ms),
                    "launches": launches, "requests_per_layer": round(n_req, 1),
                    "gather_GBps_over_step": round(gather / (ms * 1e-3) / 1e9, 2),
                    "gather_frac_of_h2d_peak": round(gather / (ms * 1e-3) / 1e9 / h2d_peak, 3),
                    "h2d_GBps_over_step": round(h2d / (ms * 1e-3) / 1e9, 2),
                    "h2d_frac_of_h2d_peak": round(h2d / (ms * 1e-3) / 1e9 / h2d_peak, 3),
                    "gather": "capped delta: at most %d new blocks per (request, KV head) per step, zero-copy from pinned "
                              "host memory; the local blocks are appended on the GPU and never cross the link; the "
                              "committed token's K/V is written through to the host pool (counted in d2h)" % cap}
        if "mirror" in r:
            r["e2e"]["exposed_us_per_layer"] = round((ms - r["mirror"]["ms_per_step"]) * 1e3 / n, 2)
        del eng
        torch.cuda.empty_cache()
    r["_sel_gpu"] = sel_gpu
    return r


def cap_of(ratio, k):
    return max(1, int(math.floor(ratio * k)))          # Sec. 5.5.1: at most this fraction of the K selected blocks


def write_summary(path, line, rows_sweep, cells, cmd):
    """A short markdown summary of one run: the numbers the JSON line carries, as tables."""
    out = ["# %s" % line["config"]["workload"], "", "Command: `%s`" % cmd, "",
           "One B200; SM clock median %s MHz of %s, throttle reasons %s; pinned H2D peak %.1f GB/s; HBM copy peak %.1f GB/s (%s)."
           % (line["clocks"]["sm_mhz"], line["clocks"]["sm_max_mhz"], line["clocks"]["reasons"] or "none",
              line["staged"]["pinned_h2d_peak_GBps"], line["roofline"]["peak"], line["roofline"]["peak_kind"]), ""]
    if cells:
        out += ["| K blocks | drafts | cap | step in HBM ms | host-KV step ms | e2e step ms | tokens/s/layer (host KV) | fused kernel us (frac of copy peak) | recall |",
                "|---|---|---|---|---|---|---|---|---|"]
        for c in cells:
            kl = c.get("kernels", {}).get("layer", {})
            out.append("| %d | %d | %d | %s | %s | %s | %s | %s (%s) | %s |" % (
                c["k_blocks"], c["n_draft"], c["cap"], c.get("mirror", {}).get("ms_per_step"), c.get("host", {}).get("ms_per_step"),
                c.get("e2e", {}).get("ms_per_step"), c.get("host", {}).get("value"), kl.get("us"), kl.get("frac_of_measured"),
                c.get("recall_lookahead_topk")))
    else:
        v, m, e = line, line.get("value_hbm_mirror") or {}, line.get("e2e") or {}
        out += ["| quantity | value |", "|---|---|",
                "| step, full KV in pinned host memory (`value`) | %.4f ms = %.1f us/layer = %.0f tokens/s/layer |"
                % (v["ms_per_step"], v["ms_per_step"] * 1e3 / line["config"]["layers"], v["value"]),
                "| step, full KV mirrored in HBM | %s ms |" % m.get("ms_per_step"),
                "| end-to-end step (queries H2D, outputs D2H) | %s ms = %s tokens/s/layer |" % (e.get("ms_per_step"), e.get("value")),
                "| exposed transfer per layer (host-KV step - HBM step) | %s us |" % line["staged"].get("exposed_us_per_layer"),
                "| gathered bytes over the host-KV step | %s GB/s = %s of the pinned peak |"
                % (line["staged"].get("gather_GBps_over_step"), line["staged"].get("gather_frac_of_h2d_peak")),
                "| gathered bytes over the e2e step | %s GB/s = %s of the pinned peak (all H2D bytes: %s) |"
                % (e.get("gather_GBps_over_step"), e.get("gather_frac_of_h2d_peak"), e.get("h2d_frac_of_h2d_peak")),
                "| fused kernel, graph of one launch per layer | %s us = %s of the copy peak |"
                % (line["roofline"].get("us"), line["roofline"].get("frac")),
                "| fused kernel, one launch alone | %s of the copy peak |" % line["roofline"].get("frac_single_launch"),
                "| scoring + attention bytes over the HBM step | %s of the copy peak |" % line["roofline"].get("frac_in_step"),
                "| recall (lookahead vs true-query estimator) / (vs attention mass) | %s / %s |"
                % (line.get("recall_lookahead_topk"), (line.get("recall_attention_mass") or {}).get("value"))]
        if line.get("sustained"):
            su = line["sustained"]
            out.append("| host-KV step over %s s (%d replays of the timed graph) | %s ms at a median SM clock of %s MHz, reasons %s |"
                       % (su["seconds"], su["repeats"], su["ms_per_step"], su["sm_mhz_median"], su["reasons"] or "none"))
    if rows_sweep:
        out += ["", "Fetch-ratio sweep (cap = floor(ratio x K) blocks per (request, KV head) per step; exposed = step with the pool in "
                "pinned host memory minus step with the pool in HBM):", "",
                "| fetch ratio (cap) | step in HBM us/layer | host-KV us/layer | exposed us/layer | e2e us/layer | e2e exposed us/layer | "
                "gathered MB/layer | gather GB/s over host-KV step (frac of pinned peak) | e2e tokens/s/layer |",
                "|---|---|---|---|---|---|---|---|---|"]
        n = line["config"]["layers"]
        for r in rows_sweep:
            out.append("| %s (%d) | %.1f | %.1f | %.1f | %.1f | %.1f | %.2f | %.1f (%.2f) | %.0f |" % (
                r["fetch_ratio"], r["cap"], r["mirror"]["ms_per_step"] * 1e3 / n, r["host"]["ms_per_step"] * 1e3 / n,
                r["host"]["exposed_us_per_layer"], r["e2e"]["ms_per_step"] * 1e3 / n, r["e2e"]["exposed_us_per_layer"],
                r["host"]["h2d_bytes_per_step"] / n / 1e6, r["host"]["gather_GBps_over_step"],
                r["host"]["gather_frac_of_h2d_peak"], r["e2e"]["value"]))
    with open(path, "w") as f:
        f.write("\n".join(out) + "\n")


def strip_private(r):
    return {k: v for k, v in r.items() if not k.startswith("_")}


def run_ours(args):
    world, rank, local = dist_setup(args)
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    cfg, name = workload(args)
    W, K = max(args.warmup, 3), args.steps
    hbm_peak, peak_kind = measured_peaks()
    bench = Bench(args, cfg, dev, rank)
    h2d_peak = time_pinned_h2d(dev)
    bench.h2d_peak, bench.hbm_peak = h2d_peak, hbm_peak
    bench.generate(want_mirror=not args.skip_mirror, want_host=True)
    cells, rows_sweep = [], []
    if args.config == 4:
        # budget x draft-length cells; the headline cell is budget 2,048 tokens, 4 draft tokens
        for k in BUDGETS:
            for td in DRAFTS:
                w = Work(bench, k, td)
                c = measure(bench, w, world, W, K, cap_of(args.fetch_ratio, k), hbm_peak, h2d_peak,
                            want_mirror=not args.skip_mirror, want_e2e=not args.skip_e2e)
                cells.append(c)
                del w
        main = next(c for c in cells if c["k_blocks"] == 128 and c["n_draft"] == 4)
        w = Work(bench, 128, 4)
    else:
        w = Work(bench, cfg.k_blocks, cfg.n_draft)
        main = measure(bench, w, world, W, K, cap_of(args.fetch_ratio, w.k), hbm_peak, h2d_peak,
                       want_mirror=not args.skip_mirror, want_e2e=not args.skip_e2e, repeats=args.repeats)
        for tok in [t for t in args.sweep_ratios.split(",") if t]:
            ratio = float(tok)
            r = main if abs(ratio - args.fetch_ratio) < 1e-9 else \
                measure(bench, w, world, W, K, cap_of(ratio, w.k), hbm_peak, h2d_peak, want_kernels=False)
            r = dict(r)
            r["fetch_ratio"] = tok
            rows_sweep.append(r)

    cpu, recall_mass = None, None
    if rank == 0 and world == 1 and not args.skip_cpu and bench.sample_layer is not None:
        cpu, recall_mass = cpu_leg(bench, w, cfg, main.get("_sel_gpu"), main.get("_sel_step", 0))

    if rank == 0:
        host, mirror = main.get("host", {}), main.get("mirror", {})
        kern = main.get("kernels", {})
        dom = main.get("dominant", "layer")
        d = kern.get(dom, {})
        cap = main["cap"]
        line = {
            "metric": METRIC, "value": host.get("value"), "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
            "ms_per_step": host.get("ms_per_step"), "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": {"workload": "%s: batch %d, %d layers, %dq/%dkv heads, d128, context %d (+1 per step), 16-token blocks, "
                                   "budget %d tokens, %d draft tokens" % (name, cfg.batch, cfg.layers, cfg.n_q_heads, cfg.n_kv_heads,
                                                                          cfg.context, main["k_blocks"] * 16, main["n_draft"]),
                       "layers": cfg.layers, "global_batch": cfg.batch * world, "parallelism": "replicas x%d" % world,
                       "l2": "inputs larger than L2: each step streams %d layers x %.0f MB of distinct summaries + staged KV"
                             % (cfg.layers, main["algorithmic_MB_per_layer"]),
                       "kv": "full KV in pinned host memory (value, e2e); value_hbm_mirror: the same pool copied to HBM",
                       "gather": "delta selection with capped eviction, fetch ratio %.2f (cap %d blocks per head per step); local "
                                 "blocks appended on the GPU" % (args.fetch_ratio, cap),
                       "launch": "CUDA graphs of %d consecutive decode steps over 6-10 streams, instantiated and uploaded to the device "
                                 "before the timed region; a layer's attention and scoring are "
                                 "one fused launch (oasis_attn_and_score); %s gathers of %d layers per launch; side-stream "
                                 "events picked up every %d layers"
                                 % (args.group if args.group > 0 else K,
                                    args.transfer_kind or ("bulk (copy unit)" if bench.link_bound(w, cap) else "warp-per-entry"),
                                    bench.transfer_group(w, cap), bench.wait_group())},
            "gpu_launches": host.get("launches"),
            "clocks": {kk: (host.get("clocks") or {}).get(kk) for kk in ("sm_mhz", "sm_max_mhz", "reasons", "samples")},
            "roofline": {"bound": "hbm", "kernel": dom, "achieved": d.get("GBps"), "peak": hbm_peak, "unit": "GB/s",
                         "frac": d.get("frac_of_measured"), "us": d.get("us"),
                         "frac_single_launch": d.get("frac_single_launch"),
                         "frac_in_step": (main.get("step_hbm") or {}).get("frac_of_measured"),
                         "traffic": profile_traffic() if args.config == 1 and not (args.batch or args.context) else None,
                         "peak_kind": peak_kind + " (STREAM-style copy)",
                         "timing": "frac: CUDA events around a graph of one launch per layer (distinct working sets, consecutive "
                                   "launches overlap through programmatic dependent launch as in the step); frac_single_launch: "
                                   "events around one launch alone, median over the layers; frac_in_step: scoring + attention bytes "
                                   "of all layers over the whole step with the KV mirrored in HBM; traffic: dram bytes per launch "
                                   "from the tracked ncu summary of these shapes"},
            "kernels": kern,
            "recall_lookahead_topk": main.get("recall_lookahead_topk"), "recall_attention_mass": recall_mass,
            "e2e": main.get("e2e"), "cpu_baseline": cpu, "setup_seconds": round(bench.gen_seconds, 1),
            "value_hbm_mirror": mirror or None, "step_hbm": main.get("step_hbm"),
            "staged": {"pinned_h2d_peak_GBps": round(h2d_peak, 2), "requests_per_layer": host.get("requests_per_layer"),
                       "gather_GBps_over_step": host.get("gather_GBps_over_step"),
                       "gather_frac_of_h2d_peak": host.get("gather_frac_of_h2d_peak"),
                       "exposed_us_per_layer": host.get("exposed_us_per_layer"),
                       "compute_to_host_step_ratio": host.get("compute_to_host_step_ratio"),
                       "h2d_bytes_per_step": host.get("h2d_bytes_per_step"), "d2h_bytes_per_step": host.get("d2h_bytes_per_step"),
                       "ms_per_step_again": host.get("ms_per_step_again")},
        }
        if host.get("sustained"):
            line["sustained"] = host["sustained"]
        if cells:
            line["cells"] = [strip_private(c) for c in cells]
        if rows_sweep:
            line["sweep"] = [{kk: r[kk] for kk in ("fetch_ratio", "cap", "mirror", "host", "e2e") if kk in r} for r in rows_sweep]
        if args.summary:
            write_summary(args.summary, line, rows_sweep, cells, "python bench.py " + " ".join(sys.argv[1:]))
        print(json.dumps(line))


# -------------------------------------------------------------------------------------- reference


def run_reference(args):
    """The CPU oracle, as it stands, timed on this host's cores on the same workload; every
    step is a bounded sample (one request of one layer)."""
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import numpy as np
    from oracle import oracle
    oracle.lib()
    cfg, name = workload(args)
    k = 128 if args.config == 4 else cfg.k_blocks
    td = 4 if args.config == 4 else cfg.n_draft
    one = synth.scaled(cfg, batch=1, layers=1, steps=1, n_draft=td)
    lay = synth.make_layer(one, seed=args.seed, layer=0, device="cpu")
    kv = synth.u16(lay.host_kv)
    table, n_full, seq = lay.block_table.numpy(), lay.n_full.numpy(), lay.seq_len.numpy()
    q = synth.u16(lay.q)
    summ = oracle.build_summaries(kv, table, np.zeros(1, np.int32), n_full)

    def one_step():
        s32, _ = oracle.score_blocks(q[:, 1:], summ, n_full)
        sel, idx, slots = oracle.select_topk(s32, n_full, seq, one.n_q_tokens, k, table)
        pool = np.zeros((one.n_kv_heads * (k + 2), 2, 16, 128), np.uint16)
        oracle.stage_blocks(kv.reshape(-1, 2, 16, 128), idx, slots, pool)
        oracle.sparse_attn(q, pool, slots.reshape(1, one.n_kv_heads, -1), sel, seq,
                           np.float32(1.0 / math.sqrt(128.0)), one.n_kv_heads)

    W, K = max(args.warmup, 1), args.steps
    for _ in range(W):
        one_step()
    t0 = time.perf_counter()
    for _ in range(K):
        one_step()
    dt = (time.perf_counter() - t0) / K
    value = 1.0 / dt                     # one request through one layer per sample
    sample = "each step = 1 request x 1 layer of the workload (score+top-k+gather+attention), single thread"
    line = {"impl": "reference", "metric": METRIC, "value": round(value, 3), "unit": UNIT, "n_gpus": world,
            "steps": K, "warmup": W, "ms_per_step": round(dt * 1e3, 3), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": "%s (bounded sample): %s" % (name, sample)},
            "cpu_baseline": {"value": round(value, 3), "unit": UNIT, "cores": 1, "host_cores": os.cpu_count(), "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": round(value, 3), "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


if __name__ == "__main__":
    a = parse_args()
    if a.impl == "reference":
        run_reference(a)
    else:
        run_ours(a)
