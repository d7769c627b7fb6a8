#!/usr/bin/env python
"""Benchmark of the draft-tree verification step (one JSON line on stdout).

A *step* is one pass of the whole hot path over one batch of synthetic input:
    vispec_tree_mask_build -> vispec_tree_verify_attn x L layers (each layer its own cache buffers)
    -> vispec_accept_commit (acceptance + commit over all L layers in one launch).
`value` is verify-attention KV GB/s: the K and V bytes the L attention calls must read
(sum_b 2*(S_b+N)*Hkv*D*2 per layer) divided by the whole step's device time.  Inputs are resident in
HBM before the timed region; the L layers' caches total far more than L2, so no flush is needed.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config llava7b] [--impl reference]

With N > 1 (torchrun, one rank per GPU) every rank runs an independent replica of the workload: the
path has no exchange step, so there is no collective on the data path; `value` sums the replicas.
`--impl reference` times the CPU fp64 oracle on the host cores instead (rank 0 only).
"""
from __future__ import annotations

import argparse
import ctypes
import json
import math
import os
import subprocess
import sys
import tempfile
import threading
import time
from concurrent.futures import ThreadPoolExecutor

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "verify-attention KV GB/s (tree-verify step: mask + L x attention + accept + compact)"
FALLBACK_HBM_GBS = 6650.0
# DRAM bytes (read + write) of one attention launch, per workload, from an ncu capture of that launch
# (dram__bytes_read.sum + dram__bytes_write.sum, two launches averaged).  A figure is only valid for the kernel it was
# taken on: set an entry to None when the attention kernel changes and take the counters again.
NCU_TRAFFIC_BYTES_PER_LAUNCH = {
    "llava7b": 66_180_000,                # 65.58 MB read + 0.61 MB written
    "llava13b_b4": 335_860_000,           # 330.23 MB read + 5.63 MB written
    "qwen3b_S32768_N16_B8": 274_060_000,  # attention launch only (270.09 + 3.97 MB); the merge kernel is its own launch
    "qwen3b_S8192_N60_B4": 35_150_000,    # four row blocks per kv head share their tiles through L2
    "qwen7b": 7_580_000,                  # seven row blocks per kv head share their tiles through L2
}
FALLBACK_BF16_TFLOPS = 1400.0             # sustained figure of the fallback measurement
EXP_PER_CLK_PER_SM = 16                   # special-function lanes of one SM (4 per scheduler)
# Workloads timed briefly after the headline (attention sweep only), each against its own binding roofline.
OTHER_WORKLOADS = [("qwen7b", 28, False, 0), ("llava13b_b4", 8, False, 0), ("llava13b_b4", 8, False, 16),
                   ("qwen3b_S8192_N16_B4", 16, False, 0), ("qwen3b_S8192_N60_B4", 16, False, 0), ("llava7b", 8, True, 0)]


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--config", default="llava7b")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--layers", type=int, default=0, help="use only the first LAYERS layers (profiling captures)")
    ap.add_argument("--split-form", type=int, default=0, help="VISPEC_OPT_SPLIT_FORM of the context (0 automatic; see vispec.h)")
    ap.add_argument("--no-others", action="store_true", help="skip the short timed runs of the other workloads")
    ap.add_argument("--no-sampled", action="store_true", help="skip the timing of vispec_accept_sampled")
    ap.add_argument("--paged", type=int, default=0, help="serve the caches from a block pool of this many slots per block (16/32/64/128)")
    ap.add_argument("--token-major", action="store_true", help="with --paged: pool blocks are [slots, kv heads, D] instead of [kv heads, slots, D]")
    ap.add_argument("--with-rope", action="store_true", help="also run vispec_rope_tree_rows before each layer's attention")
    ap.add_argument("--fused-rope", action="store_true", help="with --with-rope: one table per step and vispec_tree_verify_attn_rope per layer instead of two calls")
    ap.add_argument("--no-graph", action="store_true", help="launch every kernel from Python instead of replaying graphs")
    return ap.parse_args()


def measured_peaks():
    """(HBM GB/s, sustained bf16 TFLOP/s, max SM MHz, "measured" | "fallback")."""
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return (float(d["hbm_gbs"]), float(d.get("bf16_tflops_sustained", FALLBACK_BF16_TFLOPS)),
                float(d.get("sm_max_mhz", 1965.0)), "measured")
    return FALLBACK_HBM_GBS, FALLBACK_BF16_TFLOPS, 1965.0, "fallback"


def attention_roofline(cfg, kv_len, us_per_launch, sm_count, traffic=None):
    """The roofline of one attention launch: the time each resource needs for the launch's algorithmic work - K and V
    rows from HBM (512 B per cached token per kv head at D = 128), the two contractions on the tensor cores
    (4*D*G*N flops per cached token per kv head, against the sustained bf16 figure: the launch sits inside a long
    step) and the softmax's exponentials on the special-function units (G*N per cached token per kv head) - names
    the largest as the bound and reports the achieved rate against that resource's peak."""
    hbm_gbs, tflops, sm_mhz, kind = measured_peaks()
    tokens = int(sum(int(s) + cfg.N for s in kv_len)) * cfg.Hkv          # cached tokens x kv heads
    kv_bytes = tokens * 4 * cfg.D
    flops = tokens * 4 * cfg.D * cfg.G * cfg.N
    exps = tokens * cfg.G * cfg.N
    exp_peak = EXP_PER_CLK_PER_SM * sm_count * sm_mhz * 1e6               # exponentials per second
    t = {"hbm": kv_bytes / (hbm_gbs * 1e9), "tensor": flops / (tflops * 1e12), "alu": exps / exp_peak}
    bound = max(t, key=t.get)
    sec = us_per_launch * 1e-6
    if bound == "hbm":
        achieved, peak, unit = kv_bytes / sec / 1e9, hbm_gbs, "GB/s"
    elif bound == "tensor":
        achieved, peak, unit = flops / sec / 1e12, tflops, "TFLOP/s"
    else:
        achieved, peak, unit = exps / sec / 1e12, exp_peak / 1e12, "Texp/s"
    return {"bound": bound, "achieved": achieved, "peak": peak, "unit": unit, "frac": achieved / peak,
            "peak_kind": f"of {kind}", "floor_us": {k: v * 1e6 for k, v in t.items()},
            "kv_gbs": kv_bytes / sec / 1e9, "pct_of_8TBs": 100.0 * kv_bytes / sec / 8e12, "traffic": traffic}


# ------------------------------------------------------------------------------------ rank logic

def max_over_ranks(values, world, device="cpu"):
    """Element-wise maximum of a list of floats over all ranks (identity for a single process)."""
    if world <= 1:
        return [float(v) for v in values]
    import torch
    import torch.distributed as dist
    t = torch.tensor(values, dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t]


def whole_job_gbs(bytes_per_replica_step, steps, seconds, world):
    """Whole-job throughput of `world` independent replicas that all finished `steps` steps within `seconds`."""
    return world * bytes_per_replica_step * steps / seconds / 1e9


# ------------------------------------------------------------------------------------ clocks

class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.out = open(self.path, "w")
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu), f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "50"], stdout=self.out, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        res = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return res
        try:
            self.proc.terminate()
            self.proc.wait(timeout=5)
            self.out.close()
            rows = [l.strip().split(", ") for l in open(self.path) if l.strip()]
            os.unlink(self.path)
            sm = [float(r[0]) for r in rows if len(r) >= 7]
            power = [float(r[2]) for r in rows if len(r) >= 7]
            if sm:
                busy = [s for s, p in zip(sm, power) if p >= 0.5 * max(power)] or sm
                res["sm_mhz"] = float(np.median(busy))
                res["sm_max_mhz"] = float(rows[0][1])
                res["power_w_max"] = max(power)
                res["samples"] = len(sm)
                names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
                for j, n in enumerate(names):
                    if any(r[3 + j].strip().lower().startswith("active") for r in rows if len(r) >= 7):
                        res["reasons"].append(n)
        except Exception:
            pass
        return res


# ------------------------------------------------------------------------------------ workload

def build_host_inputs(cfg, layers):
    """Seeded host inputs for all layers (numpy, bf16 bit patterns); generation is threaded."""
    from paper_2509_15235_b200 import synth
    tree = synth.make_tree_inputs(cfg)
    with ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 1)) as ex:
        per_layer = list(ex.map(lambda l: synth.make_layer_tensors(cfg, l), range(layers)))
    return tree, per_layer


class DeviceWorkload:
    """All device buffers of one replica plus the step function that drives the C ABI."""

    def __init__(self, cfg, tree, per_layer, device):
        import torch
        from paper_2509_15235_b200 import binding
        self.torch, self.cfg = torch, cfg
        self.L = len(per_layer)
        dev = torch.device("cuda", device)
        self.dev = dev
        B, N, Hq, Hkv, D = cfg.B, cfg.N, cfg.Hq, cfg.Hkv, cfg.D
        self.ctx = binding.VerifyContext(B, N, Hq, Hkv, D, cfg.S_max, self.L, device=device)

        def bf16(bits):
            return torch.from_numpy(bits.view(np.int16)).to(dev).view(torch.bfloat16)

        def i32(a):
            return torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(dev)

        self.k = [bf16(x["k_cache"]) for x in per_layer]
        self.v = [bf16(x["v_cache"]) for x in per_layer]
        self.q = torch.stack([bf16(x["q"]) for x in per_layer])            # [L,B,N,Hq,D]
        self.out = torch.zeros_like(self.q)
        for l in range(self.L):
            self.ctx.cache_register(l, self.k[l], self.v[l])
        self.parents, self.draft, self.target = i32(tree["parents"]), i32(tree["draft_ids"]), i32(tree["target_ids"])
        self.kv_len = i32(tree["kv_len"])
        W = (N + 63) // 64
        self.mask = torch.zeros((B, N, W), dtype=torch.int64, device=dev)
        self.depth = torch.zeros((B, N), dtype=torch.int32, device=dev)
        self.path = torch.zeros((B, N), dtype=torch.int32, device=dev)
        self.alen = torch.zeros(B, dtype=torch.int32, device=dev)
        self.bonus = torch.zeros(B, dtype=torch.int32, device=dev)
        self.new_len = torch.zeros(B, dtype=torch.int32, device=dev)
        self.scale = 1.0 / math.sqrt(D)
        self.kv_bytes_per_layer = cfg.kv_bytes_per_layer(tree["kv_len"])
        self.with_rope = False
        self.page_rows = 0

    def enable_rope(self, tree, theta):
        """Also rotate the tree rows and write them into the cache before each layer's attention (the step that
        precedes it in a decoder layer).  The rows fed in are seeded noise; positions are kv_len + depth."""
        torch, cfg = self.torch, self.cfg
        g = torch.Generator(device=self.dev).manual_seed(1234)
        shape = (self.L, cfg.B, cfg.N, cfg.Hkv, cfg.D)
        self.k_new = torch.randn(shape, generator=g, device=self.dev, dtype=torch.float32).to(torch.bfloat16)
        self.v_new = torch.randn(shape, generator=g, device=self.dev, dtype=torch.float32).to(torch.bfloat16)
        self._pre()
        torch.cuda.synchronize()
        self.positions = (self.kv_len[:, None] + self.depth).to(torch.int32).contiguous()
        self.theta = theta
        self.with_rope = True
        self.fused_rope = False
        self.rope_table = self.ctx.rope_table_build(self.positions, theta)

    def enable_paging(self, page_rows, token_major=False):
        """Re-home every layer's cache in a block pool [num_blocks, Hkv, page_rows, D] with the blocks in a seeded
        random order (what a serving stack's allocator leaves behind) and serve the step through the *_paged calls."""
        torch, cfg = self.torch, self.cfg
        B, Hkv, S_max, D = self.k[0].shape
        per = S_max // page_rows
        g = torch.Generator(device="cpu").manual_seed(4321)
        perm = torch.randperm(B * per, generator=g).to(self.dev)
        self.block_table = perm.view(B, per).to(torch.int32).contiguous()
        for l in range(self.L):
            pools = []
            for c in (self.k[l], self.v[l]):
                blocks = c.view(B, Hkv, per, page_rows, D).permute(0, 2, 1, 3, 4).reshape(B * per, Hkv, page_rows, D)
                pool = torch.empty(blocks.shape, dtype=blocks.dtype, device=blocks.device)
                pool[perm] = blocks
                pools.append(pool.permute(0, 2, 1, 3).contiguous() if token_major else pool)
            self.k[l], self.v[l] = pools
            self.ctx.cache_register_paged(l, self.k[l], self.v[l], token_major)
        self.page_rows = page_rows

    def _pre(self):
        self.ctx.tree_mask_build(self.parents, self.mask, self.depth)
        if self.with_rope and getattr(self, "fused_rope", False):
            self.ctx.rope_table_build(self.positions, self.theta, self.rope_table)      # once per cycle, for every layer

    def _attn(self):
        for l in range(self.L):
            if self.with_rope and self.fused_rope and not self.page_rows:
                self.ctx.tree_verify_attn_rope(l, self.q[l], self.k_new[l], self.v_new[l], self.rope_table, self.kv_len,
                                               self.mask, self.scale, self.out[l])
                continue
            if self.with_rope and self.page_rows:
                self.ctx.rope_tree_rows_paged(l, self.q[l], self.k_new[l], self.v_new[l], self.positions, self.kv_len,
                                              self.block_table, self.theta)
            elif self.with_rope:
                self.ctx.rope_tree_rows(l, self.q[l], self.k_new[l], self.v_new[l], self.positions, self.kv_len,
                                        self.theta)
            if self.page_rows:
                self.ctx.tree_verify_attn_paged(l, self.q[l], self.kv_len, self.block_table, self.mask, self.scale,
                                                self.out[l])
            else:
                self.ctx.tree_verify_attn(l, self.q[l], self.kv_len, self.mask, self.scale, self.out[l])

    def _probe(self):
        for l in range(self.L):
            self.ctx.stream_probe(l, self.kv_len, self.cfg.N)

    def _post(self):
        # acceptance and commit in one launch; kv_len itself is left as it was so that every step sees the same workload
        if self.page_rows:
            self.ctx.accept_commit_paged(0, self.L, self.draft, self.target, self.parents, self.kv_len, self.block_table,
                                         self.path, self.alen, self.bonus, self.new_len)
            return
        self.ctx.accept_commit(0, self.L, self.draft, self.target, self.parents, self.kv_len, self.path, self.alen,
                               self.bonus, self.new_len)

    def capture(self):
        """Capture the three phases of a step as CUDA graphs (the launches are the same C-ABI calls;
        replaying them removes the Python/ctypes time between launches from the device timeline)."""
        torch = self.torch
        self.graphs = []
        for fn in (self._pre, self._attn, self._post):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                fn()
            self.graphs.append(g)
        self.launches_per_step = None

    def step(self, ev_attn=None):
        if getattr(self, "graphs", None):
            pre, attn, post = (g.replay for g in self.graphs)
        else:
            pre, attn, post = self._pre, self._attn, self._post
        pre()
        if ev_attn:
            ev_attn[0].record()
        attn()
        if ev_attn:
            ev_attn[1].record()
        post()


class HostStep:
    """End-to-end step: the cycle's inputs start in pinned host memory and its results end there.
    Per step: H2D of parents / draft_ids / target_ids / kv_len, of q for all layers and of the tree's
    new K/V rows for all layers; D2H of the attention output of all layers, the accepted path, accept_len,
    bonus and the new kv_len.  The committed prefix of the cache is state that lives on the device across cycles.
    The layers go in four groups: while one group's attention runs, the next group's inputs arrive on a second
    stream and the previous group's outputs leave on a third (PCIe carries both directions at once).  The tree's
    rows are put behind the committed prefix by vispec_rope_tree_rows with all positions 0 (the identity rotation:
    the synthetic rows stand for rows that are already rotated)."""

    GROUPS = 4

    def __init__(self, wl: DeviceWorkload, tree, per_layer):
        torch = wl.torch
        self.wl = wl
        cfg = wl.cfg
        pin = lambda t: t.pin_memory()
        self.h_q = pin(wl.q.cpu())
        self.h_out = pin(torch.zeros_like(self.h_q))
        S = tree["kv_len"]
        N = cfg.N
        # new rows [L,B,N,Hkv,D] gathered from the synthetic caches (host side, outside the timed region)
        rows_k = np.stack([np.stack([x["k_cache"][b, :, S[b]:S[b] + N].transpose(1, 0, 2) for b in range(cfg.B)]) for x in per_layer])
        rows_v = np.stack([np.stack([x["v_cache"][b, :, S[b]:S[b] + N].transpose(1, 0, 2) for b in range(cfg.B)]) for x in per_layer])
        self.h_newk = pin(torch.from_numpy(np.ascontiguousarray(rows_k).view(np.int16)).view(torch.bfloat16))
        self.h_newv = pin(torch.from_numpy(np.ascontiguousarray(rows_v).view(np.int16)).view(torch.bfloat16))
        self.d_newk = torch.empty_like(self.h_newk, device=wl.dev)
        self.d_newv = torch.empty_like(self.h_newv, device=wl.dev)
        self.h_ints = pin(torch.from_numpy(np.concatenate([tree["parents"].ravel(), tree["draft_ids"].ravel(),
                                                           tree["target_ids"].ravel(), tree["kv_len"].ravel()]).astype(np.int32)))
        self.d_ints = torch.empty_like(self.h_ints, device=wl.dev)
        BN = cfg.B * N
        self.views = (self.d_ints[:BN].view(cfg.B, N), self.d_ints[BN:2 * BN].view(cfg.B, N),
                      self.d_ints[2 * BN:3 * BN].view(cfg.B, N), self.d_ints[3 * BN:])
        self.d_res = torch.zeros(BN + 3 * cfg.B, dtype=torch.int32, device=wl.dev)
        self.h_res = pin(torch.zeros(BN + 3 * cfg.B, dtype=torch.int32))
        self.pos0 = torch.zeros((cfg.B, N), dtype=torch.int32, device=wl.dev)
        self.h2d = (self.h_q.numel() + self.h_newk.numel() + self.h_newv.numel()) * 2 + self.h_ints.numel() * 4
        self.d2h = self.h_out.numel() * 2 + self.h_res.numel() * 4
        g = max(1, min(self.GROUPS, wl.L))
        edges = [round(i * wl.L / g) for i in range(g + 1)]
        self.groups = [(edges[i], edges[i + 1]) for i in range(g) if edges[i + 1] > edges[i]]
        self.s_in, self.s_out = torch.cuda.Stream(device=wl.dev), torch.cuda.Stream(device=wl.dev)
        self.ev_in = [torch.cuda.Event() for _ in self.groups]
        self.ev_done = [torch.cuda.Event() for _ in self.groups]

    def step(self):
        wl, cfg = self.wl, self.wl.cfg
        torch = wl.torch
        B, N = cfg.B, cfg.N
        main = torch.cuda.current_stream()
        self.s_in.wait_stream(main)                 # the previous step has let go of the input buffers
        with torch.cuda.stream(self.s_in):
            for i, (lo, hi) in enumerate(self.groups):
                wl.q[lo:hi].copy_(self.h_q[lo:hi], non_blocking=True)
                self.d_newk[lo:hi].copy_(self.h_newk[lo:hi], non_blocking=True)
                self.d_newv[lo:hi].copy_(self.h_newv[lo:hi], non_blocking=True)
                self.ev_in[i].record(self.s_in)
        self.d_ints.copy_(self.h_ints, non_blocking=True)
        parents, draft, target, kv_len = self.views
        c = wl.ctx
        path = self.d_res[:B * N].view(B, N)
        alen, bonus, new_len = self.d_res[B * N:B * N + B], self.d_res[B * N + B:B * N + 2 * B], self.d_res[B * N + 2 * B:]
        c.tree_mask_build(parents, wl.mask, wl.depth)
        for i, (lo, hi) in enumerate(self.groups):
            main.wait_event(self.ev_in[i])
            for l in range(lo, hi):
                c.rope_tree_rows(l, wl.q[l], self.d_newk[l], self.d_newv[l], self.pos0, kv_len, 1e4)   # placement
                c.tree_verify_attn(l, wl.q[l], kv_len, wl.mask, wl.scale, wl.out[l])
            self.ev_done[i].record(main)
            self.s_out.wait_event(self.ev_done[i])
            with torch.cuda.stream(self.s_out):
                self.h_out[lo:hi].copy_(wl.out[lo:hi], non_blocking=True)
        c.accept_commit(0, wl.L, draft, target, parents, kv_len, path, alen, bonus, new_len)
        self.h_res.copy_(self.d_res, non_blocking=True)
        main.synchronize()                           # the caller reads accept_len to go on
        self.s_out.synchronize()


def time_other_workload(name, layers, redundant, device, min_seconds=0.4, page_rows=0):
    """Attention sweep of one further workload (L layers, each its own cache pair, graph replay), timed for at least
    `min_seconds` with the clocks sampled meanwhile, against that workload's own binding roofline.  Trees and
    lengths come from the seeded generators; q/K/V are N(0,1) bf16 drawn on the device (timing only: these
    workloads have their parity tests).  `redundant`: the image span of every head repeats one key (Sec. 4.1, Eq. 2).
    `page_rows`: the caches are pools of blocks of that many slots, addressed through a block table in random order."""
    import torch
    from paper_2509_15235_b200 import binding, synth
    cfg = synth.get_config(name)
    tree = synth.make_tree_inputs(cfg)
    dev = torch.device("cuda", device)
    L = min(layers, cfg.layers)
    B, N, Hq, Hkv, D = cfg.B, cfg.N, cfg.Hq, cfg.Hkv, cfg.D
    ctx = binding.VerifyContext(B, N, Hq, Hkv, D, cfg.S_max, L, device=device)
    g = torch.Generator(device=dev).manual_seed(cfg.config_id)
    ks, vs = [], []
    for l in range(L):
        k = torch.randn((B, Hkv, cfg.S_max, D), generator=g, device=dev, dtype=torch.bfloat16)
        v = torch.randn((B, Hkv, cfg.S_max, D), generator=g, device=dev, dtype=torch.bfloat16)
        if redundant:
            k[:, :, :cfg.n_image] = k[:, :, :1]
        if page_rows:
            k = k.view(B * (cfg.S_max // page_rows), page_rows, Hkv, D).permute(0, 2, 1, 3).contiguous()    # [blocks, Hkv, rows, D]
            v = v.view(B * (cfg.S_max // page_rows), page_rows, Hkv, D).permute(0, 2, 1, 3).contiguous()
            ctx.cache_register_paged(l, k, v, False)
        else:
            ctx.cache_register(l, k, v)
        ks.append(k); vs.append(v)
    q = torch.randn((L, B, N, Hq, D), generator=g, device=dev, dtype=torch.bfloat16)
    out = torch.empty_like(q)
    i32 = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(dev)
    kv_len, parents = i32(tree["kv_len"]), i32(tree["parents"])
    mask = torch.zeros((B, N, (N + 63) // 64), dtype=torch.int64, device=dev)
    ctx.tree_mask_build(parents, mask)
    scale = 1.0 / math.sqrt(D)

    block_table = None
    if page_rows:
        per = cfg.S_max // page_rows
        perm = torch.randperm(B * per, generator=torch.Generator(device="cpu").manual_seed(4321))
        block_table = perm.view(B, per).to(torch.int32).to(dev).contiguous()

    def sweep():
        for l in range(L):
            if page_rows:
                ctx.tree_verify_attn_paged(l, q[l], kv_len, block_table, mask, scale, out[l])
            else:
                ctx.tree_verify_attn(l, q[l], kv_len, mask, scale, out[l])

    n0 = ctx.launch_count()
    sweep()
    torch.cuda.synchronize()
    launches_per_call = (ctx.launch_count() - n0) // L
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        sweep()
    for _ in range(5):
        graph.replay()
    torch.cuda.synchronize()
    sampler = ClockSampler(device)
    sampler.start()
    time.sleep(0.15)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    reps, ms = 0, 0.0
    while ms < min_seconds * 1e3:
        chunk = max(20, reps)
        e0.record()
        for _ in range(chunk):
            graph.replay()
        e1.record()
        torch.cuda.synchronize()
        ms += e0.elapsed_time(e1)
        reps += chunk
    clocks = sampler.stop()
    status = ctx.status_poll()
    us = ms * 1e3 / (reps * L)
    sm_count = torch.cuda.get_device_properties(dev).multi_processor_count
    res = attention_roofline(cfg, tree["kv_len"], us, sm_count, NCU_TRAFFIC_BYTES_PER_LAUNCH.get(name) if not (redundant or page_rows) else None)
    res.update({"workload": name + ("+redundant_image_keys" if redundant else "") + (f"+paged{page_rows}" if page_rows else ""),
                "layers": L, "us_per_layer": us,
                "sweeps": reps, "launches_per_call": launches_per_call, "status_word": status,
                "kv_mb_per_layer": cfg.kv_bytes_per_layer(tree["kv_len"]) / 1e6,
                "clocks": {k: clocks.get(k) for k in ("sm_mhz", "sm_max_mhz", "reasons", "samples", "power_w_max")}})
    ctx.close()
    del ks, vs, q, out
    torch.cuda.empty_cache()
    return res


# ------------------------------------------------------------------------------------ oracle legs

def oracle_sample(cfg, tree, layers, budget_heads):
    """Time the oracle, as it stands, on the given layers restricted to `budget_heads` kv heads (all
    of their query heads, all nodes, the full cache length) plus mask, acceptance and commit."""
    import oracle
    G = cfg.G
    hk = min(cfg.Hkv, budget_heads)
    t0 = time.perf_counter()
    mask, _, _ = oracle.tree_mask(tree["parents"])
    path, alen, _ = oracle.accept(tree["draft_ids"], tree["target_ids"], tree["parents"])
    outs = []
    for x in layers:
        q, k, v = x["q"][:, :, :hk * G], x["k_cache"][:, :hk], x["v_cache"][:, :hk]
        outs.append(oracle.tree_attn(q, k, v, tree["kv_len"], mask, 1.0 / math.sqrt(cfg.D), want_lse=False)[0])
        oracle.kv_compact(k, v, path, alen, tree["kv_len"])
    dt = time.perf_counter() - t0
    kv_bytes = len(layers) * int(sum(2 * (int(s) + cfg.N) * hk * cfg.D * 2 for s in tree["kv_len"]))
    oracle_sample.last = {"outs": outs, "accept_len": alen, "heads": hk * G}
    return kv_bytes / dt / 1e9, dt, hk, oracle.num_threads()


def run_reference(args):
    """The reference arm is the CPU oracle timed on the host cores (there is no reference code)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2509_15235_b200 import synth
    cfg = synth.get_config(args.config)
    tree = synth.make_tree_inputs(cfg)
    layer0 = [synth.make_layer_tensors(cfg, 0)]
    heads = min(cfg.Hkv, 8)
    for _ in range(min(args.warmup, 2)):
        oracle_sample(cfg, tree, layer0, heads)
    t0 = time.perf_counter()
    vals = [oracle_sample(cfg, tree, layer0, heads) for _ in range(args.steps)]
    total = time.perf_counter() - t0
    gbs = float(np.mean([v[0] for v in vals]))
    sample = (f"per step: 1 of {cfg.layers} layers, {vals[0][2]} of {cfg.Hkv} kv heads, all nodes, full KV length, "
              f"plus mask/accept/commit; fp64 C + OpenMP")
    line = {
        "impl": "reference", "metric": METRIC, "value": gbs, "unit": "GB/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / max(args.steps, 1),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": cfg.name, "note": "CPU oracle on host cores; bounded sample of the workload"},
        "cpu_baseline": {"value": gbs, "unit": "GB/s", "cores": vals[0][3], "kind": "oracle", "sample": sample},
        "e2e": {"value": gbs, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ------------------------------------------------------------------------------------ main arm

def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
        return
    import torch
    import torch.distributed as dist
    from paper_2509_15235_b200 import synth

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    torch.cuda.set_device(local)
    cfg = synth.get_config(args.config)
    warmup = max(args.warmup, 3)

    tree, per_layer = build_host_inputs(cfg, args.layers if args.layers > 0 else cfg.layers)
    wl = DeviceWorkload(cfg, tree, per_layer, local)
    if args.split_form:
        from paper_2509_15235_b200 import binding
        wl.ctx.ctx_set_option(binding.OPT_SPLIT_FORM, args.split_form)
    L = wl.L
    if args.paged:
        wl.enable_paging(args.paged, args.token_major)
    if args.with_rope:
        wl.enable_rope(tree, 1e6 if cfg.name.startswith("qwen") else 1e4)
        wl.fused_rope = bool(args.fused_rope)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident timing ----
    launches0 = wl.ctx.launch_count()
    wl.step()                                   # plain launches once: counts the kernels of one step
    torch.cuda.synchronize()
    launches_per_step = wl.ctx.launch_count() - launches0
    if not args.no_graph:
        wl.capture()
    for _ in range(warmup):
        wl.step()
    barrier()
    assert wl.ctx.status_poll() == 0
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record()
    for s in range(args.steps):
        wl.step(evs[s])
    e1.record()
    barrier()
    ms_total = e0.elapsed_time(e1)
    attn_ms = sum(a.elapsed_time(b) for a, b in evs)
    launches = launches_per_step * args.steps
    # The roofline figure: at least max(steps, 100) further attention sweeps (the L attention calls of a step, graph
    # replay, events on the launching stream) and at least half a second of them, so that the clock sampler sees the
    # load.  `value` and `ms_per_step` stay on the `steps` whole steps timed above.
    sweep_reps, sweep_ms = 0, 0.0
    if not args.no_graph:
        r0, r1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        while sweep_reps < max(args.steps, 100) or sweep_ms < 500.0:
            chunk = max(args.steps, 100)
            r0.record()
            for _ in range(chunk):
                wl.graphs[1].replay()
            r1.record()
            torch.cuda.synchronize()
            sweep_ms += r0.elapsed_time(r1)
            sweep_reps += chunk
        launches += sweep_reps * (launches_per_step - 2)
    barrier()
    clocks = sampler.stop() if rank == 0 else None
    status = wl.ctx.status_poll()
    if sweep_reps == 0:
        sweep_reps, sweep_ms = args.steps, attn_ms

    ms_total, attn_ms = max_over_ranks([ms_total, attn_ms], world, "cuda")   # (the roofline sweep is rank 0's own)
    kv_bytes_step = wl.kv_bytes_per_layer * L
    value = whole_job_gbs(kv_bytes_step, args.steps, ms_total * 1e-3, world)

    # ---- streaming-read probe: the same K/V rows through the same TMA rings, no arithmetic (context for the roofline) ----
    read_probe = None
    if rank == 0 and cfg.D == 128 and cfg.B <= 32 and not args.paged:
        torch = wl.torch
        g = torch.cuda.CUDAGraph()
        wl._probe()
        torch.cuda.synchronize()
        with torch.cuda.graph(g):
            wl._probe()
        for _ in range(3):
            g.replay()
        n_probe = max(3, min(args.steps, 50))
        r0, r1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        r0.record()
        for _ in range(n_probe):
            g.replay()
        r1.record()
        torch.cuda.synchronize()
        us = r0.elapsed_time(r1) * 1e3 / (n_probe * L)
        read_probe = {"value": wl.kv_bytes_per_layer / (us * 1e-6) / 1e9, "unit": "GB/s", "us_per_layer": us,
                      "what": "vispec_stream_probe: the K/V rows of one attention call through the same TMA rings, "
                              "nothing computed, one launch per layer"}

    # ---- the step after the forward at temperature > 0: sampled acceptance on probability rows [B,N,V] ----
    sampled = None
    if rank == 0 and not args.no_sampled:
        from paper_2509_15235_b200 import synth as _synth
        si = _synth.make_sampled_inputs(tree["parents"], cfg.vocab, 777)
        f32 = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(wl.dev)
        # 8 input sets in rotation so that the probability rows come from HBM, not from L2
        sets = [(f32(si["p_target"]), f32(si["p_draft"])) for _ in range(max(2, min(8, int(1.2e9 // si["p_target"].nbytes))))]
        ids_d = torch.from_numpy(si["draft_ids"]).to(wl.dev)
        ua_d, ub_d = f32(si["u_accept"]), f32(si["u_bonus"])
        g = torch.cuda.CUDAGraph()
        call = lambda pt, ph: wl.ctx.accept_sampled(ids_d, wl.parents, pt, ph, ua_d, ub_d, wl.path, wl.alen, wl.bonus)
        call(*sets[0])
        torch.cuda.synchronize()
        with torch.cuda.graph(g):
            for pt, ph in sets:
                call(pt, ph)
        for _ in range(3):
            g.replay()
        n_rep = 20
        r0, r1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        r0.record()
        for _ in range(n_rep):
            g.replay()
        r1.record()
        torch.cuda.synchronize()
        sampled = {"us_per_call": r0.elapsed_time(r1) * 1e3 / (n_rep * len(sets)), "vocab": cfg.vocab,
                   "accept_len": [int(x) for x in wl.alen.cpu()],
                   "what": "vispec_accept_sampled on synthetic probability rows [B,N,V] fp32, "
                           f"{len(sets)} input sets in rotation, graph replay"}
        assert wl.ctx.status_poll() == 0
        # the step before the forward: rerank of a depth-3, width-8 expansion down to N - 1 draft tokens
        K = min(cfg.N - 1, 127)
        width = 8
        rdepth = max(3, -(-(K - width) // (width * width)) + 1)
        rc = _synth.make_rerank_candidates(cfg.B, rdepth, width, cfg.vocab, 778)
        cp_d, ct_d = (torch.from_numpy(rc[k]).to(wl.dev) for k in ("cand_parent", "cand_token"))
        cs_d = f32(rc["cand_score"])
        rp = torch.zeros((cfg.B, K + 1), dtype=torch.int32, device=wl.dev)
        ri = torch.zeros_like(rp)
        rs = torch.zeros((cfg.B, K), dtype=torch.int32, device=wl.dev)
        g2 = torch.cuda.CUDAGraph()
        wl.ctx.tree_rerank(cp_d, ct_d, cs_d, K, rp, ri, rs)
        torch.cuda.synchronize()
        with torch.cuda.graph(g2):
            for _ in range(8):
                wl.ctx.tree_rerank(cp_d, ct_d, cs_d, K, rp, ri, rs)
        g2.replay()
        r0.record()
        for _ in range(n_rep):
            g2.replay()
        r1.record()
        torch.cuda.synchronize()
        sampled["tree_rerank_us_per_call"] = r0.elapsed_time(r1) * 1e3 / (n_rep * 8)
        sampled["tree_rerank_candidates"] = int(cp_d.shape[1])
        assert wl.ctx.status_poll() == 0

    # ---- end-to-end timing (host buffers in, host results out) ----
    e2e = None
    if not args.no_e2e and not args.paged:     # the host-buffer step writes the tree rows into contiguous caches
        hs = HostStep(wl, tree, per_layer)
        for _ in range(3):
            hs.step()
        barrier()
        n_e2e = max(3, min(args.steps, 20))
        t0 = time.perf_counter()
        for _ in range(n_e2e):
            hs.step()
        torch.cuda.synchronize()
        dt = time.perf_counter() - t0
        dt = max_over_ranks([dt], world, "cuda")[0]
        e2e = {"value": whole_job_gbs(kv_bytes_step, n_e2e, dt, world), "unit": "GB/s",
               "h2d_bytes_per_step": hs.h2d, "d2h_bytes_per_step": hs.d2h, "steps": n_e2e,
               "ms_per_step": 1e3 * dt / n_e2e}

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    attn_s = attn_ms * 1e-3 / (args.steps * L)               # inside the timed steps
    sweep_us = sweep_ms * 1e3 / (sweep_reps * L)             # the longer attention-only run the roofline is quoted on
    sm_count = torch.cuda.get_device_properties(local).multi_processor_count
    roof = attention_roofline(cfg, tree["kv_len"], sweep_us, sm_count,
                              NCU_TRAFFIC_BYTES_PER_LAUNCH.get(cfg.name) if not (args.paged or args.with_rope) else None)
    roof.update({"kernel": f"vispec_tree_verify_attn ({(launches_per_step - 2 - int(args.with_rope and args.fused_rope)) // L - int(args.with_rope and not args.fused_rope)} kernel launch(es) per call)",
                 "us_per_launch": sweep_us, "sweeps": sweep_reps})
    others = None
    if not args.no_others and not (args.paged or args.with_rope or args.layers):
        others = [time_other_workload(n, l, r, local, page_rows=pg) for n, l, r, pg in OTHER_WORKLOADS if not (n == cfg.name and not r and not pg)]
    line = {
        "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps, "warmup": warmup,
        "ms_per_step": ms_total / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": cfg.name, "B": cfg.B, "Hq": cfg.Hq, "Hkv": cfg.Hkv, "D": cfg.D, "N": cfg.N,
                   "kv_len": [int(s) for s in tree["kv_len"]], "layers": L,
                   "kv_bytes_per_layer": wl.kv_bytes_per_layer,
                   "l2": f"inputs larger than L2: {L} layers x {wl.kv_bytes_per_layer / 1e6:.1f} MB rotate, no flush",
                   "launch": "plain C-ABI calls" if args.no_graph else "C-ABI calls captured once, replayed as 3 CUDA graphs per step",
                   "rope_tree_rows": bool(args.with_rope), "rope_fused": bool(args.with_rope and args.fused_rope), "paged_block_rows": args.paged, "paged_token_major": bool(args.token_major),
                   "parallelism": "replicas only" if world > 1 else "single GPU"},
        "verify_steps_per_s": world * args.steps / (ms_total * 1e-3),
        "attn_us_per_layer": attn_s * 1e6,
        "pct_of_8TBs": roof["pct_of_8TBs"],
        "read_probe": read_probe,
        "around_the_forward": sampled,
        "status_word": status,
        "roofline": roof,
        "other_workloads": others,
        "clocks": clocks,
        "gpu_launches": int(launches),
    }
    if e2e:
        line["e2e"] = e2e
    if not args.no_cpu_baseline:
        n_l = L
        gbs, dt, hk, cores = oracle_sample(cfg, tree, per_layer[:n_l], cfg.Hkv)
        if e2e:
            # the last end-to-end step's host-side results against what the oracle has just computed from the same inputs
            ref = oracle_sample.last
            got = hs.h_out.float().numpy()
            err = max(float(np.abs(got[l][:, :, :ref["heads"]] - o).max()) for l, o in enumerate(ref["outs"]))
            got_len = hs.h_res[cfg.B * cfg.N:cfg.B * cfg.N + cfg.B].numpy()
            if err > 2e-2 or not np.array_equal(got_len, ref["accept_len"]):
                raise RuntimeError(f"end-to-end results differ from the oracle: max abs err {err}, accept_len {got_len}")
            e2e["checked_against_oracle"] = {"layers": len(ref["outs"]), "max_abs_err": err}
        line["cpu_baseline"] = {"value": gbs, "unit": "GB/s", "cores": cores, "kind": "oracle",
                                "sample": f"one step: {n_l} of {L} layers, {hk} of {cfg.Hkv} kv heads, all nodes, full KV "
                                          f"length, plus mask/accept/commit ({dt:.1f} s of fp64 C + OpenMP)"}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
