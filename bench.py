#!/usr/bin/env python
"""Benchmark of the dynamic-vocabulary path (LZW update + hyper-encoder + joint logits).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

One "step" of a decode workload is one z2z_decode_step over its batch of B sequences: joint
logits and selection, online LZW update with the selected code, hyper-encoder on the new entry of
each sequence for both caches.  The prompts are compressed and their entries embedded before the
timed region (session set-up).  The default workload is the Llama-3-8B-shaped head, the largest
decode configuration that fits one GPU; with no `--workload` given on one GPU the same JSON line
also carries a `per_workload` object with the other bf16 configurations (Phi-3-mini-shaped head,
long context, and the prompt-scoring configuration at its full 64 prompts), each with its own step
time, roofline figures, end-to-end figure and clocks.  Prints ONE JSON line.

Timed regions.  A region is EXACTLY K steps between two CUDA events, bracketed by a barrier and a
device synchronise.  A decode step takes a fraction of a millisecond, so when K steps cover less
than 0.3 s the region is repeated (on fresh hidden states, the session simply goes on decoding)
until that much time is covered; `ms_per_step` and `value` are those of the MEDIAN region, the
spread is reported beside them, and the clock sampler runs over all of them.

`--impl reference` times the CPU oracle (oracle/) as it stands on the host cores, on a bounded
sample of the same workload.  With `--gpus N` each of N ranks runs an independent replica of the
workload (the path has no exchange step); times are the maximum over ranks, token counts the sum.
When the launcher's environment (WORLD_SIZE) is absent, `--gpus N` starts the N ranks itself.
"""
from __future__ import annotations

import argparse
import gc
import json
import math
import os
import socket
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2506_01084_b200 import synth_inputs as si  # noqa: E402

METRIC = "base-token-equiv decode tok/s (LZW+hyper-embed+logits)"
UNIT = "base tokens/s"
DEFAULT_WORKLOAD = "llama3_8b_head"
SUB_WORKLOADS = ("phi3_mini_head", "long_context", "prefill_heavy")
MIN_TIMED_S = 0.3            # a K-step region is repeated until this much device time is covered
MAX_REGIONS = 200


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        j = json.load(open(p))
        return {"hbm_gbs": float(j["hbm_gbs"]), "bf16_tflops": float(j["bf16_tflops"]),
                "bf16_tflops_sustained": float(j.get("bf16_tflops_sustained", j["bf16_tflops"])),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0,
            "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and clock-event (throttle) reasons through NVML, the library nvidia-smi
    itself reads, from a thread while the timed region runs (nvidia-smi's own loop cannot sample
    faster than its start-up time, and a timed region lasts a fraction of a second).
    Reading only: nothing is set."""

    def __init__(self, index: int, period_s: float = 0.004):
        self.index, self.period, self.samples = index, period_s, []
        self._stop = threading.Event()
        self.thread, self.err = None, None

    def start(self):
        try:
            import pynvml
            pynvml.nvmlInit()
            vis = os.environ.get("CUDA_VISIBLE_DEVICES")
            idx = self.index
            if vis:
                ent = [v.strip() for v in vis.split(",") if v.strip()][idx]
                self.h = (pynvml.nvmlDeviceGetHandleByIndex(int(ent)) if ent.isdigit()
                          else pynvml.nvmlDeviceGetHandleByUUID(ent))
            else:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(idx)
            self.nv = pynvml
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception as e:                      # no NVML: report that instead of clocks
            self.err = f"NVML unavailable: {type(e).__name__}"
            return
        self.thread = threading.Thread(target=self._run, daemon=True)
        self.thread.start()

    def _run(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                mhz = nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)
                rs = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                pw = nv.nvmlDeviceGetPowerUsage(self.h) / 1000.0
                self.samples.append((float(mhz), int(rs), pw))
            except Exception:
                pass
            time.sleep(self.period)

    def stop(self):
        if self.thread is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [self.err or "not sampled"]}
        self._stop.set()
        self.thread.join(timeout=2)
        nv = self.nv
        names = {"hw_slowdown": nv.nvmlClocksEventReasonHwSlowdown,
                 "hw_thermal_slowdown": nv.nvmlClocksEventReasonHwThermalSlowdown,
                 "sw_thermal_slowdown": nv.nvmlClocksEventReasonSwThermalSlowdown,
                 "sw_power_cap": nv.nvmlClocksEventReasonSwPowerCap}
        reasons = sorted(k for k, bit in names.items() if any(r & bit for _, r, _ in self.samples))
        sm = [m for m, _, _ in self.samples if m > 0]
        return {"sm_mhz": float(np.median(sm)) if sm else None,
                "sm_mhz_min": float(min(sm)) if sm else None, "sm_max_mhz": self.max_mhz,
                "reasons": reasons, "samples": len(sm),
                "power_w_max": max((p for _, _, p in self.samples), default=None)}


# --------------------------------------------------------------------------------------------------
# algorithmic bytes of one decode step (what the kernels must move at minimum)
# --------------------------------------------------------------------------------------------------
def logits_bytes(w: si.Workload, n_hyper_total: float) -> float:
    """W_U once + every visible hyper-unembedding row once + hidden rows (bf16 = 2 B)."""
    es = 2 if w.dtype == "bf16" else 4
    return es * (w.V * w.d + n_hyper_total * w.d + w.B * w.d)


def encoder_gemm_bytes(w: si.Workload) -> float:
    """Linear-layer weights of both hyper-encoders, each streamed once per step."""
    es = 2 if w.dtype == "bf16" else 4
    per_layer = 4 * w.d * w.d + 2 * w.d * w.dff
    return es * per_layer * w.enc_layers * (1 if w.tied else 2)


def replica_seed(rank: int) -> int:
    """Seed of a rank's replica of the workload: ranks run independent replicas (different token
    streams, weights and hidden states), the path has no exchange step between sequences."""
    return 1000 + rank


def reduce_over_ranks(times_ms, counts, world: int, device):
    """Whole-job numbers from per-rank ones: every time becomes the MAX over ranks, every count
    the SUM over ranks.  The only collectives of the benchmark (the data path has none)."""
    if world <= 1:
        return list(times_ms), list(counts)
    tt = torch.tensor(list(times_ms), device=device, dtype=torch.float64)
    torch.distributed.all_reduce(tt, op=torch.distributed.ReduceOp.MAX)
    cc = torch.tensor(list(counts), device=device, dtype=torch.float64)
    torch.distributed.all_reduce(cc, op=torch.distributed.ReduceOp.SUM)
    return tt.tolist(), cc.tolist()


def plan_regions(K: int, est_ms_per_step: float, steps_available: int, min_s: float = MIN_TIMED_S) -> int:
    """Number of K-step regions: enough to cover `min_s` of device time at the estimated step
    time, at most what the session's remaining codebook room (in steps) allows, at least one."""
    want = int(math.ceil(1.1 * min_s * 1e3 / max(K * est_ms_per_step, 1e-6)))    # 10 % over: the estimate is a probe
    room = max(1, steps_available // max(K, 1))
    return max(1, min(want, room, MAX_REGIONS))


# --------------------------------------------------------------------------------------------------
# synthetic inputs shared between the workloads of one run (same seed and shape -> same tensor)
# --------------------------------------------------------------------------------------------------
class Inputs:
    """Generated weights, kept on the host and on the device and keyed by what determines their
    values, so that workloads with the same table and encoder shapes do not draw (or upload) them
    again: three of the configurations share V and d and differ only in the position table."""

    def __init__(self, dev):
        self.dev, self.host, self.gpu = dev, {}, {}

    def tables(self, w, seed):
        key = ("tables", w.V, w.d, w.dtype, w.tied, seed)
        if key not in self.host:
            self.host[key] = si.make_tables(w, seed)
        return self.host[key]

    def encoder(self, w, seed):
        key = ("enc", w.d, w.dff, w.enc_layers, w.dtype, seed)
        if key not in self.host:
            self.host[key] = si.make_encoder(w, seed)             # pos belongs to this w.M
            self.host[key + ("M",)] = w.M
        if self.host[key + ("M",)] == w.M:
            return self.host[key]
        # same seed and shapes except pos[M, d]: only that tensor is drawn again (tensor i of the
        # list depends on the seed and on i alone); kept, so that its device copy stays valid
        pkey = key + ("pos", w.M)
        if pkey not in self.host:
            self.host[pkey] = si.normal_tensor((w.M, w.d), 0.02, seed * 131 + 0, w.torch_dtype)
        return [self.host[pkey]] + list(self.host[key][1:])

    def to_dev(self, t):
        key = (t.data_ptr(), tuple(t.shape))
        if key not in self.gpu:
            self.gpu[key] = t.to(self.dev)
        return self.gpu[key]


def forced_codes(zb, w, cb, dev, stream, prompt_code_lens, n_steps: int):
    """Teacher forcing: the codes a zip2zip model would have to emit to continue each sequence
    with the generator's own tokens.  The whole stream (prompt + continuation) is compressed in a
    scratch session; by the online property of LZW its first k - 1 codes are the first k - 1 codes
    of the prompt alone (k = the prompt's code count; the prompt's last code is a flush that the
    longer stream may extend).  The session `cb` is restarted and grown from those k - 1 codes, so
    that it is in exactly the state in which the stream's k-th, k+1-th ... codes are the next
    ones.  Returns them as [n_steps, B] int32 on the device."""
    cfg = zb.make_config(w.V, 8, w.M, w.cap, w.B, "fp32", 0, 1, 8)
    scratch = zb.Codebook(cfg, dev)
    T_full = stream.shape[1]
    codes = torch.zeros(w.B, T_full, dtype=torch.int32, device=dev)
    clen = torch.zeros(w.B, dtype=torch.int32, device=dev)
    zb.z2z_lzw_encode(scratch, torch.from_numpy(stream).to(dev), None, codes, clen, None)
    k = (prompt_code_lens.clamp(min=1) - 1).to(torch.int32)    # codes replayed per sequence
    if int((clen - k).min().item()) < n_steps:
        raise SystemExit("the continuation is too short for the requested steps")
    zb.z2z_codebook_init(cb)                                    # new session on the same handle
    toks = torch.zeros(w.B, w.T + 8, dtype=torch.int32, device=dev)
    tlen = torch.zeros(w.B, dtype=torch.int32, device=dev)
    zb.z2z_lzw_decode(cb, codes, k, zb.DECODE_REPLAY, toks, tlen)
    idx = k.to(torch.int64)[None, :] + torch.arange(n_steps, device=dev)[:, None]      # [n_steps, B]
    forced = torch.gather(codes.t().contiguous(), 0, idx).to(torch.int32).contiguous()
    torch.cuda.synchronize()
    del scratch
    return forced


def kernel_source_digest() -> str:
    """Digest of the code of the streaming kernels (comments and blank space left out); an ncu
    traffic figure only counts while it matches the code that produced it."""
    import hashlib
    import re
    h = hashlib.sha256()
    d = os.path.join(ROOT, "paper_2506_01084_b200", "csrc")
    for f in ("z2z_stream.cu", "z2z_stream.h", "z2z_sm100.cuh", "z2z_decode_logits.cu"):
        with open(os.path.join(d, f), "r") as fh:
            text = fh.read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        text = re.sub(r"//[^\n]*", "", text)
        h.update(" ".join(text.split()).encode())
    return h.hexdigest()[:12]


def ncu_traffic(kernel_class: str, workload: str):
    """DRAM bytes per launch (read + write) of a kernel class from the committed ncu summary
    profiles/dram_traffic.txt, or None when there is no figure for the present kernel sources.
    Line format:  class workload source-digest bytes-per-launch"""
    path = os.path.join(ROOT, "profiles", "dram_traffic.txt")
    if not os.path.exists(path):
        return None
    dig = kernel_source_digest()
    for ln in open(path):
        f = ln.split("#")[0].split()
        if len(f) >= 4 and f[0] == kernel_class and f[1] == workload and f[2] == dig:
            return float(f[3])
    return None


def _local_device():
    dev = torch.device(f"cuda:{int(os.environ.get('LOCAL_RANK', 0))}")
    torch.cuda.set_device(dev)
    return dev


def _barrier(world):
    if world > 1:
        torch.distributed.barrier()
    torch.cuda.synchronize()


# --------------------------------------------------------------------------------------------------
# decode workloads
# --------------------------------------------------------------------------------------------------
def run_decode(args, w: si.Workload, inputs: Inputs, rank: int, world: int):
    from paper_2506_01084_b200 import binding as zb
    zb.lib()                                  # fail loudly if the CUDA library is missing
    dev = inputs.dev
    K, Wm = args.steps, args.warmup
    Ka = min(K, 128)                          # steps of the per-kernel, end-to-end and sampling passes
    seed = replica_seed(rank)
    forced_mode = args.decode_mode == "forced"
    n_probe = 8
    # hidden states for every step that may run: regions are planned after the warm-up, bounded here
    # (a step cannot be faster than its algorithmic bytes at 8 TB/s, which bounds the steps 0.3 s can hold)
    floor_s = (logits_bytes(w, 0) + encoder_gemm_bytes(w)) / 8e12
    max_steps = Wm + n_probe + 3 * Ka + min(K * MAX_REGIONS, int(MIN_TIMED_S / floor_s) + 2 * K, max(K, int(w.cap)))
    if forced_mode:
        stream = si.make_tokens(w, seed, T=w.T + max_steps * w.M + 64)
        tokens = np.ascontiguousarray(stream[:, :w.T])
    else:
        stream = None
        tokens = si.make_tokens(w, seed)
    W_E, W_U = inputs.tables(w, seed)
    encE_t = [inputs.to_dev(t) for t in inputs.encoder(w, seed * 3 + 1)]
    encU_t = encE_t if w.tied else [inputs.to_dev(t) for t in inputs.encoder(w, seed * 3 + 2)]
    g_WE = inputs.to_dev(W_E)
    g_WU = g_WE if w.tied else inputs.to_dev(W_U)
    cfg = zb.make_config(w.V, w.d, w.M, w.cap, w.B, w.dtype, w.enc_layers, w.heads, w.dff, w.tied)
    cb = zb.Codebook(cfg, dev)
    encE, encU = zb.encoder_weights(encE_t), zb.encoder_weights(encU_t)
    E_h = torch.zeros(w.B, w.cap, w.d, dtype=w.torch_dtype, device=dev)
    U_h = E_h if w.tied else torch.zeros_like(E_h)
    hidden_host = si.make_hidden(w, max_steps * w.B, seed).view(max_steps, w.B, w.d).pin_memory()
    hidden = hidden_host.to(dev)

    # ---- session set-up (not timed as steps; reported separately) ----
    g_tok = torch.from_numpy(tokens).to(dev)
    codes = torch.zeros(w.B, w.T, dtype=torch.int32, device=dev)
    clen = torch.zeros(w.B, dtype=torch.int32, device=dev)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
    torch.cuda.synchronize()
    ev[0].record()
    zb.z2z_lzw_encode(cb, g_tok, None, codes, clen, None)
    ev[1].record()
    n_codes = int(clen.sum().item())           # a prompt creates fewer entries than it has codes
    ev[3].record()
    zb.z2z_hyper_embed(cb, zb.CACHE_EMBED, g_WE, encE, None, None, n_codes, E_h, None)
    if not w.tied:
        zb.z2z_hyper_embed(cb, zb.CACHE_UNEMBED, g_WU, encU, None, None, n_codes, U_h, None)
    ev[2].record()
    torch.cuda.synchronize()
    forced_dev = None
    if forced_mode:
        forced_dev = forced_codes(zb, w, cb, dev, stream, clen, max_steps)
        # the session now holds the codebook of the prompt's codes but the last (replayed from the
        # stream's own codes, so that the continuation's codes name its entries): embed them again
        E_h.zero_(); U_h.zero_()
        zb.z2z_hyper_embed(cb, zb.CACHE_EMBED, g_WE, encE, None, None, w.B * w.T, E_h, None)
        if not w.tied:
            zb.z2z_hyper_embed(cb, zb.CACHE_UNEMBED, g_WU, encU, None, None, w.B * w.T, U_h, None)
        torch.cuda.synchronize()
    st, n0 = zb.z2z_status(cb)
    _, setup_launches = zb.z2z_profile_read(cb)
    prefill = {"lzw_encode_ms": ev[0].elapsed_time(ev[1]), "hyper_embed_all_ms": ev[3].elapsed_time(ev[2]),
               "prompt_tokens": int(w.B * w.T), "compressed_tokens": int(clen.sum().item()),
               "hypertokens": int(n0.sum().item()),
               "launches": setup_launches,
               "note": "session set-up, not part of the timed steps; z2z_hyper_embed is given max_entries = "
                       "the prompts' code count, which bounds its passes of 1024 entries"}

    nxt_all = torch.zeros(max_steps, w.B, dtype=torch.int32, device=dev)
    lse = torch.zeros(w.B, dtype=torch.float32, device=dev)
    cursor = [0]                               # next unused step (hidden row block, sampling step)

    def step(t, select=None):
        zb.z2z_decode_step(cb, hidden[t], g_WE, g_WU, encE, encU, E_h, U_h,
                           zb.SELECT_ARGMAX if select is None else select, 1.0, 0, t,
                           None if forced_dev is None else forced_dev[t], nxt_all[t], None, lse)

    def run_steps(n, select=None):
        t0 = cursor[0]
        for t in range(t0, t0 + n):
            step(t, select)
        cursor[0] = t0 + n
        return t0

    def timed(n, select=None):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        _barrier(world)
        e0.record()
        t0 = run_steps(n, select)
        e1.record()
        _barrier(world)
        return e0.elapsed_time(e1), t0

    run_steps(Wm)
    est_ms, _ = timed(n_probe)
    est_ms /= n_probe
    # room: every step may add one entry per sequence; once all codebooks are full the encoder
    # pass is no longer launched and a step is a different (cheaper) thing
    _, n_now = zb.z2z_status(cb)
    room_steps = int(w.cap - int(n_now.max().item())) - 3 * Ka - 1
    room_steps = min(room_steps, max_steps - cursor[0] - 3 * Ka)
    R = plan_regions(K, est_ms, room_steps, args.min_timed_s)
    if world > 1:                              # every rank runs the same number of regions
        rr = torch.tensor([R], device=dev, dtype=torch.int64)
        torch.distributed.all_reduce(rr, op=torch.distributed.ReduceOp.MIN)
        R = int(rr.item())
    zb.z2z_profile_read(cb)                    # reset launch counters

    # ---- device-timed regions: inputs resident in HBM ----
    sampler = ClockSampler(dev.index or 0)
    sampler.start()
    n_before = zb.z2z_status(cb)[1].sum().item()
    regions = []
    for _ in range(R):
        ms, t0 = timed(K)
        regions.append((ms, t0))
    clocks = sampler.stop()
    _, launches = zb.z2z_profile_read(cb)
    launches = {k: v / R for k, v in launches.items()}          # per K-step region
    n_after = zb.z2z_status(cb)[1].sum().item()

    # ---- Ka steps again with per-kernel-class events (for the roofline numbers) ----
    zb.z2z_profile(cb, True)
    run_steps(Ka)
    zb.z2z_profile(cb, False)
    cls_ms, cls_launches = zb.z2z_profile_read(cb)
    n_after2 = zb.z2z_status(cb)[1].sum().item()

    # ---- end to end: host buffers, H2D of the hidden rows and D2H of the results every step ----
    out_host = torch.zeros(w.B, dtype=torch.int32).pin_memory()
    lse_host = torch.zeros(w.B, dtype=torch.float32).pin_memory()
    hid_dev = torch.empty(w.B, w.d, dtype=w.torch_dtype, device=dev)
    _barrier(world)
    t_start = time.perf_counter()
    e2, e3 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e2.record()
    nx_e2e = np.zeros((Ka, w.B), dtype=np.int32)
    out_np, lse_np = out_host.numpy(), lse_host.numpy()
    out_np[:] = -1
    lse_np[:] = np.nan
    t_first = cursor[0]
    for i, t in enumerate(range(t_first, t_first + Ka)):
        zb.z2z_upload_rows(hidden_host[t], hid_dev)    # host -> device by a kernel the logits kernel overlaps
        # the applied codes and the LSE go straight into pinned host memory: the result pointers of
        # the call may be host memory that is mapped into the device's address space, so the
        # device -> host transfer of the result is the kernel's own stores
        zb.z2z_decode_step(cb, hid_dev, g_WE, g_WU, encE, encU, E_h, U_h, zb.SELECT_ARGMAX, 1.0, 0, t,
                           None if forced_dev is None else forced_dev[t], out_host, None, lse_host)
        # the caller needs the token to go on: it watches the result land in host memory instead of
        # waiting for the whole stream (the cache update of this step is still running then, and
        # the next step's launches queue up behind it)
        t_wait = time.perf_counter()
        while (out_np < 0).any() or np.isnan(lse_np).any():
            if time.perf_counter() - t_wait > 5.0:
                raise RuntimeError("decode step result did not arrive in host memory")
        nx_e2e[i] = out_np
        out_np[:] = -1
        lse_np[:] = np.nan
    cursor[0] = t_first + Ka
    torch.cuda.current_stream().synchronize()
    e3.record()
    _barrier(world)
    e2e_ms = max(e2.elapsed_time(e3), (time.perf_counter() - t_start) * 1e3)

    # ---- the same step with Gumbel-max sampling instead of argmax (Section 2.3 step 9) ----
    smp_ms, smp_t0 = timed(Ka, zb.SELECT_GUMBEL)

    # ---- base-token equivalents of what was emitted ----
    stt, n_fin = zb.z2z_status(cb)
    lens = []
    for b in range(w.B):
        _, ln = zb.z2z_codebook_read(cb, b)
        lens.append(ln.numpy())
    nx = nxt_all.cpu().numpy()

    def base_tokens(zs):
        tot = 0
        for b in range(w.B):
            z = zs[:, b]
            tot += int(np.where(z < w.V, 1, lens[b][np.clip(z - w.V, 0, w.cap - 1)]).sum())
        return tot

    order = sorted(range(R), key=lambda i: regions[i][0])
    med = order[(R - 1) // 2]                                    # the median region (lower one of two)
    dev_ms, t_med = regions[med]
    bt_dev = base_tokens(nx[t_med:t_med + K])
    bt_e2e = base_tokens(nx_e2e)
    bt_smp = base_tokens(nx[smp_t0:smp_t0 + Ka])
    bad = int(sum(1 for s in stt.tolist() if s & (zb.ST_BAD_TOKEN | zb.ST_TABLE_FULL | zb.ST_WAIT_TIMEOUT)))
    all_ms = [r[0] for r in regions]

    # ---- reduce over ranks: max time, summed tokens ----
    (dev_ms, e2e_ms, smp_ms, ms_min, ms_max), (bt_dev, bt_e2e, bt_smp) = reduce_over_ranks(
        [dev_ms, e2e_ms, smp_ms, min(all_ms), max(all_ms)], [bt_dev, bt_e2e, bt_smp], world, dev)

    pk = peaks()
    es = 2 if w.dtype == "bf16" else 4
    step_input_bytes = es * (w.V * w.d + 2 * w.enc_layers * (4 * w.d * w.d + 2 * w.d * w.dff))
    l2_note = ("per-step inputs (W_U and both encoders' weights) exceed the 126 MB L2" if step_input_bytes > 126e6 else
               "per-step inputs (%.1f MB) fit the 126 MB L2 and are not flushed between steps: a small parity "
               "configuration, not a benchmark one" % (step_input_bytes / 1e6))
    mean_hyper = 0.5 * (n_after + n_after2)     # hyper rows visible during the profiled pass
    classes = {"logits": logits_bytes(w, mean_hyper), "encoder_gemm": encoder_gemm_bytes(w)}
    dom = max(classes, key=lambda k: cls_ms.get(k, 0.0))

    def class_roof(k):
        n_launch = max(cls_launches[k], 1)
        ms_launch = cls_ms[k] / n_launch                     # average launch duration
        by_launch = classes[k] * Ka / n_launch               # algorithmic bytes per launch
        gbs = by_launch / max(ms_launch, 1e-9) / 1e6
        return {"algorithmic_bytes_per_launch": by_launch, "launches_per_step": n_launch / Ka,
                "us_per_launch": ms_launch * 1e3, "ms_per_step": cls_ms[k] / Ka, "gbs": gbs,
                "frac": gbs / pk["hbm_gbs"], "traffic": ncu_traffic(k, w.name)}

    cr = {k: class_roof(k) for k in classes}
    step_bytes = logits_bytes(w, 0.5 * (n_before + n_after)) + encoder_gemm_bytes(w)
    roof = {"bound": "hbm", "kernel": {"logits": "k_decode_logits", "encoder_gemm": "k_stream_gemm"}[dom],
            "achieved": cr[dom]["gbs"], "peak": pk["hbm_gbs"], "unit": "GB/s",
            "frac": cr[dom]["frac"], "traffic": cr[dom]["traffic"],
            "peak_source": pk["source"] + " (STREAM-style copy, burst)",
            "timing": "CUDA events around every launch of the kernel on the launching stream, in a "
                      "separate pass of %d steps (the events serialise the launches, which otherwise "
                      "overlap their prologues with the previous kernel); achieved = algorithmic "
                      "bytes per launch / average launch duration" % Ka,
            "per_class_ms_per_step": {k: v / Ka for k, v in cls_ms.items()},
            "logits": cr["logits"], "encoder_gemm": cr["encoder_gemm"],
            "whole_step": {"algorithmic_bytes": step_bytes, "gbs": step_bytes / (dev_ms / K) / 1e6,
                           "frac": step_bytes / (dev_ms / K) / 1e6 / pk["hbm_gbs"]}}
    line = {
        "metric": METRIC, "value": bt_dev / (dev_ms * 1e-3), "unit": UNIT, "n_gpus": world,
        "steps": K, "warmup": Wm, "ms_per_step": dev_ms / K, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": w.dtype, "data": "synthetic",
        "config": {"workload": w.name, "V": w.V, "d": w.d, "B": w.B, "prompt_tokens": w.T,
                   "M": w.M, "cap": w.cap, "enc_layers": w.enc_layers, "enc_dff": w.dff, "tied": int(w.tied),
                   "select": ("argmax computed, the update is fed the LZW codes of a generator continuation "
                              "(teacher forcing)" if forced_mode else "argmax, free-running"),
                   "replicas": world,
                   "l2": l2_note},
        "regions": {"count": R, "steps_each": K, "timed_s": sum(all_ms) * 1e-3,
                    "ms_per_step_median": dev_ms / K, "ms_per_step_min": ms_min / K,
                    "ms_per_step_max": ms_max / K,
                    "note": "value and ms_per_step are those of the median region"},
        "steps_per_s": K / (dev_ms * 1e-3),
        "mean_phrase_len": bt_dev / (K * w.B * world),
        "new_entries_in_timed_regions": int(n_after - n_before),
        "status_errors": bad,
        "prefill": prefill,
        "e2e": {"value": bt_e2e / (e2e_ms * 1e-3), "unit": UNIT, "ms_per_step": e2e_ms / Ka, "steps": Ka,
                "h2d_bytes_per_step": int(w.B * w.d * es), "d2h_bytes_per_step": int(w.B * 8)},
        "select_gumbel": {"value": bt_smp / (smp_ms * 1e-3), "unit": UNIT, "ms_per_step": smp_ms / Ka,
                          "steps": Ka, "temperature": 1.0,
                          "vs_argmax_step": (smp_ms / Ka) / (dev_ms / K)},
        "gpu_launches": int(round(sum(launches.values()))),
        "gpu_launches_by_class": launches,
        "clocks": clocks,
        "roofline": roof,
    }
    del cb, E_h, U_h, hidden, nxt_all
    return line


# --------------------------------------------------------------------------------------------------
# oracle on the host cores (cpu_baseline of our arm, and the whole `--impl reference` arm)
# --------------------------------------------------------------------------------------------------
def oracle_sample(w: si.Workload, n_steps: int, seed: int = 1000, prompt_tokens: int | None = None,
                  inputs: Inputs | None = None):
    """Times `n_steps` decode steps of the oracle session on the workload's shapes.

    Bounded sample: prompts are cut to `prompt_tokens` tokens so that embedding their entries in
    fp64 stays within seconds; V, d, B, M, the encoder and the per-step work (joint logits over
    V + n_b columns, LZW update, both encoders on the new entries) are the workload's own.
    """
    from oracle import decode_step as ods
    torch.set_num_threads(os.cpu_count() or 1)
    if prompt_tokens is None:
        prompt_tokens = 256 if w.d * w.B <= 3072 * 8 else 64
    T = min(w.T, prompt_tokens)
    tokens = si.make_tokens(w, seed, T=T)
    if inputs is None:
        W_E, W_U = si.make_tables(w, seed)
        eE, eU = si.make_encoder(w, seed * 3 + 1), (None if w.tied else si.make_encoder(w, seed * 3 + 2))
    else:
        W_E, W_U = inputs.tables(w, seed)
        eE, eU = inputs.encoder(w, seed * 3 + 1), (None if w.tied else inputs.encoder(w, seed * 3 + 2))
    f = lambda t: t.double().numpy()
    encE = [f(t) for t in eE]
    encU = encE if w.tied else [f(t) for t in eU]
    s = ods.Session(w.V, w.M, w.cap, w.B, w.heads, w.dtype, f(W_E), f(W_E) if w.tied else f(W_U),
                    encE, encU)
    t0 = time.perf_counter()
    s.prefill([tokens[b].tolist() for b in range(w.B)])
    t_prefill = time.perf_counter() - t0
    hid = si.make_hidden(w, n_steps * w.B, seed).double().numpy().reshape(n_steps, w.B, w.d)
    base = 0
    t0 = time.perf_counter()
    for t in range(n_steps):
        sc, _ = s.step(hid[t], 0, 1.0, 0, t)
        base += sum(len(s.books[b].phrase(sc[b]["choice"])) for b in range(w.B))
    dt = time.perf_counter() - t0
    return {"value": base / dt, "unit": UNIT, "cores": os.cpu_count(), "kind": "oracle",
            "threads": torch.get_num_threads(),
            "sample": f"{n_steps} decode steps of the full-shape workload {w.name} (V, d, B, M, encoder as "
                      f"configured) after " + (f"prompts CUT to {T} of {w.T} tokens (a smaller codebook state than "
                      f"the GPU arm's)" if T < w.T else f"the full prompts of {T} tokens") +
                      f"; oracle prefill took {t_prefill:.1f} s; numpy fp64, {torch.get_num_threads()} threads",
            "seconds": dt, "ms_per_step": dt / n_steps * 1e3}


def run_reference(args):
    w = si.WORKLOADS[args.workload or DEFAULT_WORKLOAD]
    if w.steps == 0:
        print(json.dumps({"impl": "reference", "unavailable": "the oracle arm times decode steps; "
                          "this workload has none"}))
        return
    K = max(1, args.steps)
    per_step = 1 if w.d >= 2048 else 4
    n = max(1, min(K, 6 if w.d * w.B <= 3072 * 8 else 2)) * per_step
    res = oracle_sample(w, n_steps=n)
    line = {"impl": "reference", "metric": METRIC, "value": res["value"], "unit": UNIT,
            "n_gpus": args.gpus, "steps": K, "warmup": args.warmup,
            "ms_per_step": res["ms_per_step"], "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": w.name, "V": w.V, "d": w.d, "B": w.B, "M": w.M, "cap": w.cap},
            "cpu_baseline": {k: res[k] for k in ("value", "unit", "cores", "threads", "kind", "sample")},
            "e2e": {"value": res["value"], "unit": UNIT, "h2d_bytes_per_step": 0,
                    "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


# --------------------------------------------------------------------------------------------------
# prompt-scoring workloads (no decode steps): encode + embed every entry + logits at every position
# --------------------------------------------------------------------------------------------------
def run_prompt_scoring(args, w: si.Workload, inputs: Inputs, rank: int, world: int, K: int, Wm: int):
    """One step = the whole prompt pass of the workload: LZW encode of every prompt, hyper-encoder
    over every codebook entry for both caches, joint logits + LSE / argmax at every compressed
    position (all n_b hypertokens of the sequence visible, the paper's training convention)."""
    from paper_2506_01084_b200 import binding as zb
    zb.lib()
    dev = inputs.dev
    if args.seqs:
        w = w.scaled(B=args.seqs)
    seed = replica_seed(rank)
    tokens = si.make_tokens(w, seed)
    W_E, W_U = inputs.tables(w, seed)
    encE_t = [inputs.to_dev(t) for t in inputs.encoder(w, seed * 3 + 1)]
    encU_t = [inputs.to_dev(t) for t in inputs.encoder(w, seed * 3 + 2)]
    g_WE, g_WU = inputs.to_dev(W_E), inputs.to_dev(W_U)
    cfg = zb.make_config(w.V, w.d, w.M, w.cap, w.B, w.dtype, w.enc_layers, w.heads, w.dff, 0)
    cb = zb.Codebook(cfg, dev)
    encE, encU = zb.encoder_weights(encE_t), zb.encoder_weights(encU_t)
    E_h = torch.zeros(w.B, w.cap, w.d, dtype=w.torch_dtype, device=dev)
    U_h = torch.zeros_like(E_h)
    tok_host = torch.from_numpy(tokens).pin_memory()
    g_tok = tok_host.to(dev)
    codes = torch.zeros(w.B, w.T, dtype=torch.int32, device=dev)
    clen = torch.zeros(w.B, dtype=torch.int32, device=dev)
    # first pass fixes the number of compressed positions, so that the hidden rows can be drawn
    zb.z2z_lzw_encode(cb, g_tok, None, codes, clen, None)
    N = int(clen.sum().item())
    row_seq = torch.repeat_interleave(torch.arange(w.B, dtype=torch.int32, device=dev), clen.to(torch.int64))
    base = si.make_hidden(w, min(N, 16384), seed)
    hid_host = base[torch.arange(N) % base.shape[0]].pin_memory()      # 16384 distinct rows, repeated
    hidden = hid_host.to(dev)
    lse = torch.zeros(N, dtype=torch.float32, device=dev)
    am = torch.zeros(N, dtype=torch.int32, device=dev)
    mx = torch.zeros(N, dtype=torch.float32, device=dev)
    lse_host = torch.zeros(N, dtype=torch.float32).pin_memory()
    half_scratch = None
    if args.prompt_encoder == "fp16":
        # memory for fp16 copies of one encoder's weights: prompt-sized passes then take one
        # tensor-core pass per k-step (activations rounded once to fp16) instead of two
        nbytes = zb.encoder_half_bytes(cfg)
        half_scratch = torch.empty(nbytes + 256, dtype=torch.uint8, device=dev)
        half_scratch = half_scratch[(-half_scratch.data_ptr()) % 256:][:nbytes]
        zb.z2z_set_encoder_half_scratch(cb, half_scratch)

    def step(tok_dev, hid_dev):
        zb.z2z_codebook_init(cb)
        zb.z2z_lzw_encode(cb, tok_dev, None, codes, clen, None)
        # max_entries = -1: the call reads the entry count back (one wait on the stream) instead of
        # enqueueing a pass for every 1024 entries the prompts could have created at most
        zb.z2z_hyper_embed(cb, zb.CACHE_EMBED, g_WE, encE, None, None, -1, E_h, None)
        zb.z2z_hyper_embed(cb, zb.CACHE_UNEMBED, g_WU, encU, None, None, -1, U_h, None)
        zb.z2z_dynamic_logits(cb, hid_dev, row_seq, None, g_WU, U_h, zb.SELECT_ARGMAX, 1.0, 0, 0, None,
                              lse, am, mx)

    for _ in range(Wm):
        step(g_tok, hidden)
    zb.z2z_profile_read(cb)
    sampler = ClockSampler(dev.index or 0)
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    _barrier(world)
    e0.record()
    for _ in range(K):
        step(g_tok, hidden)
    e1.record()
    _barrier(world)
    dev_ms = e0.elapsed_time(e1)
    clocks = sampler.stop()
    _, launches = zb.z2z_profile_read(cb)
    st, n_fin = zb.z2z_status(cb)
    # per-class pass (one step: its launches run for milliseconds, the events cost nothing beside them)
    Kc = 1
    zb.z2z_profile(cb, True)
    for _ in range(Kc):
        step(g_tok, hidden)
    zb.z2z_profile(cb, False)
    cls_ms, cls_launches = zb.z2z_profile_read(cb)
    # the causal variant of the scoring call (Section 2.4: entries are created in order, so what a
    # position sees is a per-row column limit; z2z_lzw_encode's entries_after supplies it), timed alone
    after = torch.zeros(w.B, w.T, dtype=torch.int32, device=dev)
    zb.z2z_codebook_init(cb)
    zb.z2z_lzw_encode(cb, g_tok, None, codes, clen, after)
    row_nvis = after[torch.arange(w.T, device=dev)[None, :] < clen[:, None]].contiguous()
    causal_ms = []
    for _ in range(3):
        c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        c0.record()
        zb.z2z_dynamic_logits(cb, hidden, row_seq, row_nvis, g_WU, U_h, zb.SELECT_ARGMAX, 1.0, 0, 0, None,
                              lse, am, mx)
        c1.record()
        torch.cuda.synchronize()
        causal_ms.append(c0.elapsed_time(c1))
    causal_flops = 2.0 * w.d * (float(N) * w.V + float(row_nvis.to(torch.int64).sum().item()))
    # end to end: prompts and hidden rows from pinned host memory, LSE back to the host
    Ke = 1
    tok_dev = torch.empty_like(g_tok)
    hid_dev = torch.empty_like(hidden)
    _barrier(world)
    t0 = time.perf_counter()
    for _ in range(Ke):
        tok_dev.copy_(tok_host, non_blocking=True)
        hid_dev.copy_(hid_host, non_blocking=True)
        step(tok_dev, hid_dev)
        lse_host.copy_(lse, non_blocking=True)
        torch.cuda.current_stream().synchronize()
    e2e_ms = (time.perf_counter() - t0) * 1e3
    (dev_ms, e2e_ms), _ = reduce_over_ranks([dev_ms, e2e_ms], [0.0], world, dev)
    pk = peaks()
    n_rows = torch.bincount(row_seq.cpu().to(torch.int64), minlength=w.B).numpy()
    flops = 2.0 * w.d * float(sum(int(n_rows[b]) * (w.V + int(n_fin[b])) for b in range(w.B)))
    n_logit = max(cls_launches["logits"], 1)
    tfs = flops * Kc / n_logit / max(cls_ms["logits"] / n_logit, 1e-9) / 1e9
    # hyper-encoder linear layers: flop per row that carries data (rows = base tokens of all entries),
    # both encoders; the kernel executes twice that (hi and lo parts of the activations)
    enc_rows = 0
    for b in range(w.B):
        _, ln = zb.z2z_codebook_read(cb, b)
        enc_rows += int(ln.numpy()[:int(n_fin[b])].sum())
    enc_flops = 2.0 * enc_rows * w.enc_layers * 2.0 * (4 * w.d * w.d + 2 * w.d * w.dff)
    enc_tfs = enc_flops * Kc / max(cls_ms["encoder_gemm"], 1e-9) / 1e9
    passes = 1.0 if half_scratch is not None else 2.0       # tensor-core passes per k-step
    prompt_tokens = w.B * w.T * world
    bad = int(sum(1 for x in st.tolist() if x & (zb.ST_BAD_TOKEN | zb.ST_TABLE_FULL | zb.ST_WAIT_TIMEOUT)))
    es = 2
    line = {
        "metric": "prompt-scoring base tok/s (LZW encode + hyper-embed of every entry + logits/LSE at every "
                  "compressed position)",
        "value": prompt_tokens * K / (dev_ms * 1e-3), "unit": UNIT, "n_gpus": world, "steps": K, "warmup": Wm,
        "ms_per_step": dev_ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": w.dtype, "data": "synthetic",
        "config": {"workload": w.name, "V": w.V, "d": w.d, "B": w.B, "prompt_tokens": w.T, "M": w.M, "cap": w.cap,
                   "compressed_positions": N, "hypertokens": int(n_fin.sum()), "replicas": world,
                   "prompt_encoder": args.prompt_encoder,
                   "l2": "W_U, the caches and the hidden rows exceed the 126 MB L2"},
        "status_errors": bad,
        "per_class_ms_per_step": {k: v / Kc for k, v in cls_ms.items()},
        "e2e": {"value": prompt_tokens * Ke / (e2e_ms * 1e-3), "unit": UNIT, "ms_per_step": e2e_ms / Ke, "steps": Ke,
                "h2d_bytes_per_step": int(tok_host.numel() * 4 + hid_host.numel() * es),
                "d2h_bytes_per_step": int(N * 4)},
        "gpu_launches": int(sum(launches.values())), "gpu_launches_by_class": launches, "clocks": clocks,
        "roofline": {"bound": "tensor", "kernel": "k_prefill_logits", "achieved": tfs,
                     "peak": pk["bf16_tflops_sustained"], "unit": "TFLOP/s", "frac": tfs / pk["bf16_tflops_sustained"],
                     "traffic": None, "peak_source": pk["source"] + " (cuBLAS bf16, sustained)",
                     "flops_per_launch": flops * Kc / n_logit, "us_per_launch": cls_ms["logits"] / n_logit * 1e3,
                     "frac_of_burst_peak": tfs / pk["bf16_tflops"], "frac_of_nominal_2250": tfs / 2250.0,
                     "causal": {"ms": min(causal_ms), "tflops": causal_flops / min(causal_ms) / 1e9,
                                "frac": causal_flops / min(causal_ms) / 1e9 / pk["bf16_tflops_sustained"],
                                "note": "the same call with per-row visibility limits (d_row_nvis = entries that exist "
                                        "once the position's code is out), best of 3, whole call with its plan kernel"},
                     "encoder_gemm": {"kernel": "k_pair_gemm", "rows": enc_rows,
                                      "operands": "one fp16 activation operand, fp16 weight copies" if half_scratch is not None
                                                  else "bf16 hi + lo activation parts, bf16 weights",
                                      "algorithmic_tflops": enc_tfs, "executed_tflops": passes * enc_tfs,
                                      "ms_per_step": cls_ms["encoder_gemm"] / Kc,
                                      "frac_executed_of_sustained_peak": passes * enc_tfs / pk["bf16_tflops_sustained"],
                                      "note": "the two-part form issues two MMAs per k-step, so the tensor pipe "
                                              "executes twice the algorithmic flop; the fp16 form issues one"}},
    }
    del cb, E_h, U_h, hidden, hid_host, lse, am, mx, half_scratch
    return line


# --------------------------------------------------------------------------------------------------
# the calls around the hot path (decompression, embedding lookup, filtered sampling), timed alone
# --------------------------------------------------------------------------------------------------
def run_helpers(args):
    """One JSON line with device times of the helper calls at the workload's sizes: prompt
    compression, decompression (replay and resident), the mixed-stream embedding lookup and
    top-k / nucleus sampling on stored logits.  Every figure is the best of five event-timed calls
    after a warm-up call; tables and logits larger than L2 where the call is bound by HBM."""
    from paper_2506_01084_b200 import binding as zb
    zb.lib()
    dev = torch.device("cuda:0")
    torch.cuda.set_device(dev)
    w = si.WORKLOADS[args.workload or DEFAULT_WORKLOAD]
    if args.seqs:
        w = w.scaled(B=args.seqs)
    pk = peaks()

    def best_ms(fn, before=None, reps=5):
        ts = []
        for i in range(reps + 1):
            if before:
                before()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            e0.record(); fn(); e1.record()
            torch.cuda.synchronize()
            if i:
                ts.append(e0.elapsed_time(e1))
        return min(ts)

    out = {}
    cfg = zb.make_config(w.V, w.d, w.M, w.cap, w.B, w.dtype, 0, 1, 8)
    cb = zb.Codebook(cfg, dev)
    tokens = si.make_tokens(w, 1000)
    g_tok = torch.from_numpy(tokens).to(dev)
    codes = torch.zeros(w.B, w.T, dtype=torch.int32, device=dev)
    clen = torch.zeros(w.B, dtype=torch.int32, device=dev)
    ms = best_ms(lambda: zb.z2z_lzw_encode(cb, g_tok, None, codes, clen, None), before=lambda: zb.z2z_codebook_init(cb))
    out["lzw_encode"] = {"ms": ms, "ns_per_token_of_a_sequence": ms * 1e6 / w.T, "B": w.B, "T": w.T}
    toks = torch.zeros(w.B, w.T, dtype=torch.int32, device=dev)
    tlen = torch.zeros(w.B, dtype=torch.int32, device=dev)
    ms = best_ms(lambda: zb.z2z_lzw_decode(cb, codes, clen, zb.DECODE_RESIDENT, toks, tlen))
    out["lzw_decode_resident"] = {"ms": ms, "round_trip_ok": bool(torch.equal(toks, g_tok))}
    ms = best_ms(lambda: zb.z2z_lzw_decode(cb, codes, clen, zb.DECODE_REPLAY, toks, tlen),
                 before=lambda: zb.z2z_codebook_init(cb))
    out["lzw_decode_replay"] = {"ms": ms, "round_trip_ok": bool(torch.equal(toks, g_tok))}
    # embedding lookup of the compressed prompts (every code of every sequence)
    _, n_b = zb.z2z_status(cb)
    h_len = clen.cpu().numpy()
    flat = torch.cat([codes[b, :int(h_len[b])] for b in range(w.B)]).contiguous()
    seq = torch.cat([torch.full((int(h_len[b]),), b, dtype=torch.int32, device=dev) for b in range(w.B)])
    es = 2 if w.dtype == "bf16" else 4
    W_E = torch.zeros(w.V, w.d, dtype=w.torch_dtype, device=dev)
    E_h = torch.zeros(w.B, max(w.cap, 1), w.d, dtype=w.torch_dtype, device=dev)
    rows = torch.empty(flat.numel(), w.d, dtype=w.torch_dtype, device=dev)
    ms = best_ms(lambda: zb.z2z_embed_lookup(cb, flat, seq, W_E, E_h, rows))
    by = 2.0 * flat.numel() * w.d * es
    out["embed_lookup"] = {"ms": ms, "rows": int(flat.numel()), "algorithmic_bytes": by, "gbs": by / ms / 1e6,
                           "frac_of_measured_hbm": by / ms / 1e6 / pk["hbm_gbs"],
                           "note": "every output row written once and its source row read once (%.0f MB); "
                                   "source rows of frequent tokens repeat and are then served by L2, so the "
                                   "rate can exceed the HBM copy rate" % (by / 1e6)}
    # top-k / nucleus sampling on stored joint logits of one decode batch
    ld = w.V + max(w.cap, 1)
    g = torch.Generator(device="cpu"); g.manual_seed(5)
    logits = (torch.randn(w.B, ld, generator=g) * 3.0).to(dev)
    n_cols = (n_b.to(torch.int32) + w.V).to(dev)
    choice = torch.zeros(w.B, dtype=torch.int32, device=dev)
    kept = torch.zeros(w.B, dtype=torch.int32, device=dev)
    for name, k, p in (("top_k_50", 50, 1.0), ("top_p_0.9", 0, 0.9), ("top_k_50_top_p_0.9", 50, 0.9)):
        ms = best_ms(lambda: zb.z2z_sample_filtered(logits, n_cols, k, p, 0.8, 7, 3, choice, kept))
        out["sample_filtered_" + name] = {"us": ms * 1e3, "rows": w.B, "columns": int(n_cols.max().item()),
                                          "kept_mean": float(kept.float().mean().item())}
    # the joint logits of one decode batch with the reductions only, and with every logit stored
    # (what filtered sampling needs beforehand)
    hid = si.make_hidden(w, w.B, 9).to(dev)
    W_U = si.normal_tensor((w.V, w.d), 0.02, 10, w.torch_dtype).to(dev)
    lse = torch.zeros(w.B, dtype=torch.float32, device=dev)
    amax = torch.zeros(w.B, dtype=torch.int32, device=dev)
    mxl = torch.zeros(w.B, dtype=torch.float32, device=dev)
    for name, store in (("logits_reductions_only", None), ("logits_stored", logits)):
        ms = best_ms(lambda: zb.z2z_dynamic_logits(cb, hid, None, None, W_U, E_h, zb.SELECT_ARGMAX, 1.0, 0, 0, None,
                                                   lse, amax, mxl, None, None, store))
        out[name] = {"us": ms * 1e3, "rows": w.B}
    line = {"helpers": out, "config": {"workload": w.name, "V": w.V, "d": w.d, "B": w.B, "T": w.T, "M": w.M,
                                       "cap": w.cap}, "data": "synthetic",
            "peak_hbm_gbs": pk["hbm_gbs"], "peak_source": pk["source"]}
    print(json.dumps(line))


# --------------------------------------------------------------------------------------------------
# replicas: `--gpus N` without a launcher's environment starts the N ranks itself
# --------------------------------------------------------------------------------------------------
def free_port() -> int:
    with socket.socket(socket.AF_INET, socket.SOCK_STREAM) as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def launch_replicas(n: int, argv) -> int:
    """Runs this script as `n` local ranks (one process per GPU) through torch.distributed.run
    with a rendezvous on 127.0.0.1 and returns the launcher's exit code.  Rank 0 prints the line."""
    from torch.distributed.run import main as torchrun
    cmd = ["--nnodes=1", f"--nproc-per-node={n}", "--master-addr", "127.0.0.1", "--master-port",
           str(free_port()), os.path.abspath(__file__)] + list(argv)
    try:
        torchrun(cmd)
    except SystemExit as e:
        return int(e.code or 0)
    return 0


def run_stub(rank: int, world: int):
    """Launcher self-test (`--stub`): no kernel runs; every rank contributes fixed per-rank numbers
    so that a CPU test can check the launch, the rendezvous, the reduction and the single line."""
    dev = torch.device("cpu")
    (ms,), (tok,) = reduce_over_ranks([10.0 + rank], [1000.0 * (rank + 1)], world, dev)
    return {"metric": METRIC, "value": tok / (ms * 1e-3), "unit": UNIT, "n_gpus": world, "steps": 1, "warmup": 0,
            "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "stub": True,
            "config": {"workload": "stub", "replicas": world, "replica_seeds": [replica_seed(r) for r in range(world)]}}


def main(argv=None):
    argv = sys.argv[1:] if argv is None else list(argv)
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=64)
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=None, choices=list(si.WORKLOADS),
                    help="default: %s, with the other bf16 configurations as sub-records" % DEFAULT_WORKLOAD)
    ap.add_argument("--sub-workloads", default="auto", choices=["auto", "on", "off"],
                    help="auto: add the per_workload sub-records when no --workload is given and one GPU runs")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--helpers", action="store_true",
                    help="time the calls around the hot path (compression, decompression, embedding lookup, "
                         "filtered sampling) at the workload's sizes instead of the decode step")
    ap.add_argument("--decode-mode", default="free", choices=["free", "forced"],
                    help="free: the selected code feeds the codebook update; forced: the update is fed the "
                         "LZW codes of a generator continuation (the selection is still computed)")
    ap.add_argument("--seqs", type=int, default=0,
                    help="prompt-scoring workloads: use this many sequences instead of the workload's B")
    ap.add_argument("--prompt-steps", type=int, default=2,
                    help="timed steps of a prompt-scoring workload (one step is a whole prompt batch)")
    ap.add_argument("--prompt-encoder", default="fp16", choices=["fp16", "two_part"],
                    help="prompt-scoring workloads: hyper-encoder GEMM operands (fp16: one tensor-core pass per "
                         "k-step on fp16 weight copies; two_part: bf16 hi + lo activation parts, two passes)")
    ap.add_argument("--min-timed-s", type=float, default=MIN_TIMED_S,
                    help="device time the repeated K-step regions of a decode workload must cover (0: one region, "
                         "for runs under a profiler)")
    ap.add_argument("--tied", action="store_true",
                    help="decode workloads: tied embedding / unembedding tables, one hyper-encoder and one cache "
                         "for both sides (Section 2.2)")
    ap.add_argument("--stub", action="store_true", help="launcher self-test: ranks report fixed numbers, no GPU work")
    args = ap.parse_args(argv)
    args.warmup = max(args.warmup, 3)
    if args.impl == "ours" and args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(launch_replicas(args.gpus, argv))
    rank = int(os.environ.get("RANK", 0))
    world = int(os.environ.get("WORLD_SIZE", 1))
    if args.impl == "reference":
        if rank == 0:
            run_reference(args)
        return
    if args.helpers:
        if rank == 0:
            run_helpers(args)
        return
    if world > 1:
        torch.distributed.init_process_group("gloo" if args.stub else "nccl")
    if args.stub:
        line = run_stub(rank, world)
    else:
        inputs = Inputs(_local_device())
        w = si.WORKLOADS[args.workload or DEFAULT_WORKLOAD]
        if args.tied:
            w = w.scaled(tied=1)
        prompt_mode = w.steps == 0
        if prompt_mode:
            line = run_prompt_scoring(args, w, inputs, rank, world, max(1, args.prompt_steps), 3)
        else:
            line = run_decode(args, w, inputs, rank, world)
        subs = args.sub_workloads == "on" or (args.sub_workloads == "auto" and args.workload is None and world == 1)
        if subs:
            per = {}
            for name in SUB_WORKLOADS:
                if name == w.name:
                    continue
                gc.collect()
                torch.cuda.empty_cache()
                sw = si.WORKLOADS[name]
                try:
                    if sw.steps == 0:
                        per[name] = run_prompt_scoring(args, sw, inputs, rank, world, max(1, args.prompt_steps), 3)
                    else:
                        per[name] = run_decode(args, sw, inputs, rank, world)
                except Exception as e:           # a sub-record must not cost the headline line
                    per[name] = {"error": f"{type(e).__name__}: {e}"[:300]}
                    continue
                for k in ("metric", "unit", "higher_is_better", "scaling", "vs_baseline", "data", "n_gpus"):
                    if k != "metric" or sw.steps > 0:
                        per[name].pop(k, None)
            line["per_workload"] = per
        if rank == 0 and world == 1 and not args.no_cpu_baseline and not prompt_mode:
            try:
                res = oracle_sample(w, n_steps=2 if w.d >= 2048 else 16, inputs=inputs)
                line["cpu_baseline"] = {k: res[k] for k in ("value", "unit", "cores", "threads", "kind", "sample")}
            except Exception as e:
                line["cpu_baseline"] = {"error": f"{type(e).__name__}: {e}"[:300], "kind": "oracle"}
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        torch.distributed.destroy_process_group()


if __name__ == "__main__":
    main()
