#!/usr/bin/env python
"""Benchmark of the structured-tensor hot path.

One step = one pass of every call of the library over the five named synthetic workloads
(operands resident in HBM): second moment (small fp32 and large bf16), third moment, MTTKRP
on an upper-half-cube tensor, TTM on a block-diagonal tensor, and the pack / unpack calls
that feed and reconstruct them.

Metric: structured GFLOP/s = useful flops over the unique / non-zero iteration space per
second (one FMA = 2 flops, loop-invariant products counted once).  The line also carries,
per kernel, the achieved fraction of its roofline.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import workloads  # noqa: E402

METRIC = "structured GFLOP/s (unique nonzero work) and % of roofline per kernel"
UNIT = "GFLOP/s"

# fp32 FMA peak of one B200: 148 SMs x 128 FMA lanes x 2 flops x 1.965 GHz (boost clock)
FP32_PEAK_TFLOPS = 2 * 148 * 128 * 1.965e9 / 1e12
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}

# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) per launch from the ncu captures summarised
# under profiles/.  moment2_tc_pair_kernel was captured at [131072, 1024] (314.7 MB) and scaled by the
# sample count to [1048576, 1024]; the TF32 kernels were captured at the benchmark configuration.
# An entry is dropped (null) when its kernel changes after the capture.
NCU_TRAFFIC_BYTES = {"sym_moment2_large": 8 * 314.7e6, "ttm_blockdiag": 312.0e6, "mttkrp_tri": 273.5e6}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        p["source"] = "measured"
        return p
    p = dict(FALLBACK_PEAKS)
    p["source"] = "fallback"
    return p


def tri(d):
    return d * (d + 1) // 2


def tet(d):
    return d * (d + 1) * (d + 2) // 6


# --------------------------------------------------------------------------------------
# sizes, useful flops and algorithmic bytes of every call of one step
# --------------------------------------------------------------------------------------

def step_table(cfg):
    """name -> dict(flops, bytes, bound, launches).  Bytes are algorithmic: packed operands
    read once plus outputs written once."""
    c1, c2, c3, c4, c5 = (cfg[k] for k in ("moment2", "moment3", "mttkrp", "ttm", "moment2_large"))
    t = {}
    t["sym_moment2"] = dict(flops=2 * c1["N"] * tri(c1["d"]), bytes=4 * (c1["N"] * c1["d"] + tri(c1["d"])),
                            bound="alu", launches=2)
    t["unpack_tri_sym"] = dict(flops=0, bytes=4 * (tri(c1["d"]) + c1["d"] ** 2), bound="hbm", launches=1)
    t["sym_moment3"] = dict(flops=2 * c2["N"] * tet(c2["d"]) + c2["N"] * tri(c2["d"]),
                            bytes=4 * (c2["N"] * c2["d"] + tet(c2["d"])), bound="alu", launches=2)
    # tensor-core variants of the third moment (pair products made on the fly): same useful work;
    # the TF32 pipe runs at half the bf16 rate
    for kind, scale in (("tf32", 0.5), ("bf16", 1.0)):
        t["sym_moment3_" + kind] = dict(flops=t["sym_moment3"]["flops"], bytes=t["sym_moment3"]["bytes"],
                                        bound="tensor", launches=2, tensor_scale=scale)
    # fourth moment (last block of the degree-2 polynomial-regression covariance) on the first d features
    c6 = cfg["moment4"]
    simp4 = c6["d"] * (c6["d"] + 1) * (c6["d"] + 2) * (c6["d"] + 3) // 24
    t["sym_moment4_bf16"] = dict(flops=2 * c6["N"] * simp4 + c6["N"] * tri(c6["d"]),
                                 bytes=4 * (c6["N"] * c6["d"] + simp4), bound="tensor", launches=4)
    t["unpack_tet_sym"] = dict(flops=0, bytes=4 * (tet(c2["d"]) + c2["d"] ** 3), bound="hbm", launches=1)
    nnz3 = tri(c3["I"]) * c3["K"]
    t["pack_tri_x_k"] = dict(flops=0, bytes=2 * 4 * nnz3, bound="hbm", launches=1)
    # THP of the packed upper-half-cube tensor with a dense one: packed operand, gathered dense operand, packed result
    t["thp_tri_x_k"] = dict(flops=nnz3, bytes=3 * 4 * nnz3, bound="hbm", launches=1)
    t["mttkrp_tri"] = dict(flops=2 * c3["R"] * nnz3 + 2 * c3["R"] * tri(c3["I"]),
                           bytes=4 * (nnz3 + (2 * c3["I"] + c3["K"]) * c3["R"]),
                           bound=("hbm" if cfg["mttkrp_tc"] else "alu"), launches=1)
    rows4 = c4["nb"] * c4["bs"] ** 2
    t["ttm_blockdiag"] = dict(flops=2 * rows4 * c4["K"] * c4["R"],
                              bytes=4 * (rows4 * (c4["K"] + c4["R"]) + c4["K"] * c4["R"]),
                              bound=("hbm" if cfg["ttm_tc"] else "alu"), launches=1)
    d4 = c4["nb"] * c4["bs"]
    t["unpack_blockdiag"] = dict(flops=0, bytes=4 * c4["R"] * (rows4 + d4 * d4), bound="hbm", launches=1)
    nb_, kw = cfg["band"]["d"], cfg["band"]["kl"] + cfg["band"]["ku"] + 1
    t["pack_band"] = dict(flops=0, bytes=2 * 4 * nb_ * kw * cfg["band"]["inner"], bound="hbm", launches=1)
    xbytes = 2 if cfg["m2_large_dtype"] == "bf16" else 4
    t["sym_moment2_large"] = dict(flops=2 * c5["N"] * tri(c5["d"]),
                                  bytes=xbytes * c5["N"] * c5["d"] + 4 * tri(c5["d"]),
                                  bound=("tensor" if cfg["m2_large_dtype"] == "bf16" else "alu"),
                                  launches=(2 if cfg["m2_large_dtype"] == "bf16" else 1))
    t["unpack_tri_sym_large"] = dict(flops=0, bytes=4 * (tri(c5["d"]) + c5["d"] ** 2), bound="hbm", launches=1)
    return t


def roofline_us(entry, peaks):
    """Roofline time of one call inside a step: the slower of useful flops at peak and
    algorithmic bytes over the measured HBM bandwidth."""
    hbm = entry["bytes"] / (peaks["hbm_gbs"] * 1e9)
    if entry["bound"] == "tensor":
        alu = entry["flops"] / (peaks["bf16_tflops_sustained"] * entry.get("tensor_scale", 1.0) * 1e12)
    elif entry["bound"] == "hbm":
        alu = 0.0
    else:
        alu = entry["flops"] / (FP32_PEAK_TFLOPS * 1e12)
    return max(hbm, alu) * 1e6


# --------------------------------------------------------------------------------------
# clocks sampling
# --------------------------------------------------------------------------------------

class ClockSampler:
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q, "--format=csv,noheader,nounits",
                 "-lms", "50"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 6:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except ValueError:
                continue
            for n, v in zip(names, f[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(mx)), "samples": len(sm),
                "reasons": sorted(reasons)}


# --------------------------------------------------------------------------------------
# the GPU arm
# --------------------------------------------------------------------------------------

def bench_config():
    cfg = {k: dict(v) for k, v in workloads.CONFIGS.items()}
    cfg["band"] = dict(d=2048, kl=512, ku=511, inner=16)
    cfg["moment4"] = dict(N=cfg["moment3"]["N"], d=32)
    cfg["m2_large_dtype"] = "bf16"
    cfg["ttm_tc"] = True
    cfg["mttkrp_tc"] = True
    return cfg


class Workload:
    """Host (pinned) and device copies of every input of one step, and the step itself."""

    def __init__(self, cfg, device, st, torch):
        self.cfg, self.st, self.torch = cfg, st, torch
        c1, c2, c3, c4, c5 = (cfg[k] for k in ("moment2", "moment3", "mttkrp", "ttm", "moment2_large"))
        pin = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory()
        host = {}
        host["X1"] = pin(workloads.moment_input("moment2"))
        host["X2"] = pin(workloads.moment_input("moment3"))
        host["X4"] = pin(host["X2"].numpy()[:, :cfg["moment4"]["d"]])      # the first d features of the same samples
        Bp3, C3, D3 = workloads.mttkrp_inputs()
        host["C3"], host["D3"] = pin(C3), pin(D3)
        Bp4, U4 = workloads.ttm_inputs()
        host["Bp4"], host["U4"] = pin(Bp4.reshape(-1, c4["K"])), pin(U4)
        if cfg["m2_large_dtype"] == "bf16":
            bits = workloads.draw_rows_bf16(c5["N"], c5["d"], c5["dist"], workloads.SEEDS["moment2_large"])
            host["X5"] = torch.from_numpy(bits.view(np.int16)).pin_memory().view(torch.bfloat16)
        else:
            host["X5"] = pin(workloads.draw_rows(c5["N"], c5["d"], c5["dist"], workloads.SEEDS["moment2_large"]))
        band = cfg["band"]
        host["band"] = pin(workloads.draw((band["d"], band["d"], band["inner"]), "normal", 77))
        self.lay3 = st.Layout(st.ST_TRI_UPPER, c3["I"], inner=c3["K"])
        self.lay4 = st.Layout(st.ST_BLOCKDIAG, c4["nb"] * c4["bs"], inner=c4["R"], nblocks=c4["nb"], bs=c4["bs"])
        self.lay_band = st.Layout(st.ST_BAND, band["d"], inner=band["inner"], kl=band["kl"], ku=band["ku"])
        self.lay1 = st.Layout(st.ST_TRI_UPPER, c1["d"])
        self.lay2 = st.Layout(st.ST_TET, c2["d"])
        self.lay5 = st.Layout(st.ST_TRI_UPPER, c5["d"])
        # the MTTKRP operand enters the step as the dense [I,I,K] tensor (zeros where i>j)
        dev_bp3 = torch.from_numpy(Bp3).to(device)
        host["B3"] = st.st_unpack(dev_bp3.view(-1), self.lay3).cpu().pin_memory()
        del dev_bp3
        self.host = host
        self.dev = {k: torch.empty_like(v, device=device) for k, v in host.items()}
        for k in host:
            self.dev[k].copy_(host[k], non_blocking=True)
        f32 = dict(dtype=torch.float32, device=device)
        self.out = {
            "m2": torch.empty(tri(c1["d"]), **f32), "m2_dense": torch.empty(c1["d"] ** 2, **f32),
            "m3": torch.empty(tet(c2["d"]), **f32), "m3_tc": torch.empty(tet(c2["d"]), **f32), "m3_dense": torch.empty(c2["d"] ** 3, **f32),
            "Bp3": torch.empty(tri(c3["I"]) * c3["K"], **f32), "thp3": torch.empty(tri(c3["I"]) * c3["K"], **f32),
            "m4": torch.empty(cfg["moment4"]["d"] * (cfg["moment4"]["d"] + 1) * (cfg["moment4"]["d"] + 2)
                              * (cfg["moment4"]["d"] + 3) // 24, **f32), "A3": torch.empty((c3["I"], c3["R"]), **f32),
            "Ap4": torch.empty((c4["nb"] * c4["bs"] ** 2, c4["R"]), **f32),
            "A4_dense": torch.empty((c4["nb"] * c4["bs"]) ** 2 * c4["R"], **f32),
            "band_p": torch.empty(st.st_packed_elems(self.lay_band), **f32),
            "m2l": torch.empty(tri(c5["d"]), **f32), "m2l_dense": torch.empty(c5["d"] ** 2, **f32),
        }
        self.ttm_flags = st.ST_FLAG_TC_TF32 if cfg["ttm_tc"] else 0
        self.mttkrp_flags = st.ST_FLAG_TC_TF32 if cfg["mttkrp_tc"] else 0
        x5dt = st.ST_BF16 if cfg["m2_large_dtype"] == "bf16" else st.ST_F32
        wsb = max(
            st.st_workspace_bytes(st.ST_OP_SYM_MOMENT2, c1["N"], c1["d"], st.ST_F32),
            st.st_workspace_bytes(st.ST_OP_SYM_MOMENT3, c2["N"], c2["d"]),
            st.st_workspace_bytes(st.ST_OP_SYM_MOMENT3, c2["N"], c2["d"], 0, 0, st.ST_FLAG_TC_TF32),
            st.st_workspace_bytes(st.ST_OP_SYM_MOMENT3, c2["N"], c2["d"], 0, 0, st.ST_FLAG_TC_BF16),
            st.st_workspace_bytes(st.ST_OP_SYM_MOMENT4, cfg["moment4"]["N"], cfg["moment4"]["d"], 0, 0, st.ST_FLAG_TC_BF16),
            st.st_workspace_bytes(st.ST_OP_MTTKRP_TRI, c3["I"], c3["K"], c3["R"]),
            st.st_workspace_bytes(st.ST_OP_TTM_BLOCKDIAG, c4["nb"], c4["bs"], c4["K"], c4["R"], self.ttm_flags),
            st.st_workspace_bytes(st.ST_OP_SYM_MOMENT2, c5["N"], c5["d"], x5dt), 256)
        self.ws = torch.empty(wsb, dtype=torch.uint8, device=device)
        self.h2d_bytes = sum(v.numel() * v.element_size() for v in host.values())
        self.result_keys = ["m2", "m3", "A3", "Ap4", "m2l"]
        self.host_out = {k: torch.empty_like(self.out[k], device="cpu").pin_memory() for k in self.result_keys}
        self.d2h_bytes = sum(v.numel() * v.element_size() for v in self.host_out.values())

    def calls(self):
        st, d, o, c = self.st, self.dev, self.out, self.cfg
        c4 = c["ttm"]
        # The long calls come first: while the GPU works on them the host queues the short ones,
        # so that their event times are GPU time and not launch latency of the Python call path.
        return [
            ("sym_moment2_large", lambda: st.st_sym_moment2(d["X5"], out=o["m2l"], ws=self.ws)),
            ("unpack_tri_sym_large", lambda: st.st_unpack(o["m2l"], self.lay5, st.ST_FILL_SYMMETRIC,
                                                          out=o["m2l_dense"])),
            ("ttm_blockdiag", lambda: st.st_ttm_blockdiag(d["Bp4"], d["U4"], c4["nb"], c4["bs"], out=o["Ap4"],
                                                          ws=self.ws, flags=self.ttm_flags)),
            ("unpack_blockdiag", lambda: st.st_unpack(o["Ap4"].view(-1), self.lay4, out=o["A4_dense"])),
            ("pack_tri_x_k", lambda: st.st_pack(d["B3"], self.lay3, out=o["Bp3"])),
            ("mttkrp_tri", lambda: st.st_mttkrp_tri(o["Bp3"], d["C3"], d["D3"], out=o["A3"], ws=self.ws,
                                                       flags=self.mttkrp_flags)),
            ("thp_tri_x_k", lambda: st.st_thp(o["Bp3"], d["B3"], self.lay3, out=o["thp3"])),
            ("sym_moment3", lambda: st.st_sym_moment3(d["X2"], out=o["m3"], ws=self.ws)),
            ("sym_moment3_tf32", lambda: st.st_sym_moment3(d["X2"], out=o["m3_tc"], ws=self.ws,
                                                             flags=st.ST_FLAG_TC_TF32)),
            ("sym_moment3_bf16", lambda: st.st_sym_moment3(d["X2"], out=o["m3_tc"], ws=self.ws,
                                                             flags=st.ST_FLAG_TC_BF16)),
            ("sym_moment4_bf16", lambda: st.st_sym_moment4(d["X4"], out=o["m4"], ws=self.ws, flags=st.ST_FLAG_TC_BF16)),
            ("unpack_tet_sym", lambda: st.st_unpack(o["m3"], self.lay2, st.ST_FILL_SYMMETRIC, out=o["m3_dense"])),
            ("pack_band", lambda: st.st_pack(d["band"], self.lay_band, out=o["band_p"])),
            ("sym_moment2", lambda: st.st_sym_moment2(d["X1"], out=o["m2"], ws=self.ws)),
            ("unpack_tri_sym", lambda: st.st_unpack(o["m2"], self.lay1, st.ST_FILL_SYMMETRIC, out=o["m2_dense"])),
        ]

    def upload(self):
        for k, v in self.host.items():
            self.dev[k].copy_(v, non_blocking=True)

    def download(self):
        for k in self.result_keys:
            self.host_out[k].copy_(self.out[k], non_blocking=True)


def dense_controls(w, torch, reps=5):
    """Every compute kernel against the same kernel forced onto the dense, unstructured iteration
    space (ST_FLAG_DENSE_CONTROL): isolated timings with an L2 flush between repetitions.  The
    gain from structure should approach dense work / unique work."""
    st, d, o, c = w.st, w.dev, w.out, w.cfg
    c1, c2, c3, c4, c5 = (c[k] for k in ("moment2", "moment3", "mttkrp", "ttm", "moment2_large"))
    DC = st.ST_FLAG_DENSE_CONTROL
    dev = w.ws.device
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    x5dt = st.ST_BF16 if c["m2_large_dtype"] == "bf16" else st.ST_F32
    wsb = max(st.st_workspace_bytes(st.ST_OP_SYM_MOMENT2, c1["N"], c1["d"], st.ST_F32, 0, DC),
              st.st_workspace_bytes(st.ST_OP_SYM_MOMENT3, c2["N"], c2["d"], 0, 0, DC),
              st.st_workspace_bytes(st.ST_OP_SYM_MOMENT2, c5["N"], c5["d"], x5dt, 0, DC), 256)
    wsc = torch.empty(wsb, dtype=torch.uint8, device=dev)
    d4 = c4["nb"] * c4["bs"]
    lay4k = st.Layout(st.ST_BLOCKDIAG, d4, inner=c4["K"], nblocks=c4["nb"], bs=c4["bs"])
    B4_dense = st.st_unpack(d["Bp4"].view(-1), lay4k)                # 16 GiB: zeros off the diagonal blocks
    A4_dense = torch.empty((d4 * d4, c4["R"]), dtype=torch.float32, device=dev)
    pairs = {
        "sym_moment2": (lambda: st.st_sym_moment2(d["X1"], out=o["m2"], ws=w.ws),
                        lambda: st.st_sym_moment2(d["X1"], out=o["m2"], ws=wsc, flags=DC), c1["d"] ** 2 / tri(c1["d"])),
        "sym_moment3": (lambda: st.st_sym_moment3(d["X2"], out=o["m3"], ws=w.ws),
                        lambda: st.st_sym_moment3(d["X2"], out=o["m3"], ws=wsc, flags=DC), c2["d"] ** 3 / tet(c2["d"])),
        "mttkrp_tri": (lambda: st.st_mttkrp_tri(o["Bp3"], d["C3"], d["D3"], out=o["A3"], ws=w.ws, flags=w.mttkrp_flags),
                       lambda: st.st_mttkrp_tri(d["B3"], d["C3"], d["D3"], out=o["A3"], ws=w.ws,
                                                flags=w.mttkrp_flags | DC), c3["I"] ** 2 / tri(c3["I"])),
        "ttm_blockdiag": (lambda: st.st_ttm_blockdiag(d["Bp4"], d["U4"], c4["nb"], c4["bs"], out=o["Ap4"], ws=w.ws,
                                                      flags=w.ttm_flags),
                          lambda: st.st_ttm_blockdiag(B4_dense, d["U4"], c4["nb"], c4["bs"], out=A4_dense, ws=w.ws,
                                                      flags=w.ttm_flags | DC), float(c4["nb"])),
        "sym_moment2_large": (lambda: st.st_sym_moment2(d["X5"], out=o["m2l"], ws=w.ws),
                              lambda: st.st_sym_moment2(d["X5"], out=o["m2l"], ws=wsc, flags=DC),
                              c5["d"] ** 2 / tri(c5["d"])),
    }

    def timed(fn):
        for _ in range(2):
            fn()
        torch.cuda.synchronize()
        ts = []
        for _ in range(reps):
            flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); fn(); e1.record()
            torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1) * 1e3)
        return float(np.median(ts))

    out = {}
    for name, (structured, control, ideal) in pairs.items():
        a, b = timed(structured), timed(control)
        out[name] = {"structured_us": round(a, 2), "control_us": round(b, 2), "ratio": round(b / a, 3),
                     "dense_over_unique": round(ideal, 3)}
    del B4_dense, A4_dense
    return out


def moment2_sample_sweep(w, torch, reps=7):
    """The small second moment (d = 64) from the named size up to 4M samples: the named size is bound by
    launch and memory latency, the sweep shows where the kernel reaches its fp32 roofline."""
    st = w.st
    dev = w.ws.device
    d = w.cfg["moment2"]["d"]
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    out = torch.empty(tri(d), dtype=torch.float32, device=dev)
    res = []
    for N in (4096, 32768, 262144, 1048576, 4194304):
        X = torch.empty((N, d), dtype=torch.float32, device=dev).uniform_(-1.0, 1.0)
        ws = torch.empty(max(st.st_workspace_bytes(st.ST_OP_SYM_MOMENT2, N, d, st.ST_F32), 256), dtype=torch.uint8, device=dev)
        for _ in range(2):
            st.st_sym_moment2(X, out=out, ws=ws)
        ts = []
        for _ in range(reps):
            flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); st.st_sym_moment2(X, out=out, ws=ws); e1.record()
            torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1) * 1e3)
        us = float(np.median(ts))
        flops, nbytes = 2 * N * tri(d), 4 * (N * d + tri(d))
        roof = max(flops / (FP32_PEAK_TFLOPS * 1e12), nbytes / (load_peaks()["hbm_gbs"] * 1e9)) * 1e6
        res.append({"N": N, "us": round(us, 2), "tflops": round(flops / us / 1e6, 2), "gbs": round(nbytes / us / 1e3, 1),
                    "roofline_us": round(roof, 2), "frac": round(roof / us, 4)})
        del X, ws
    return res


def max_over_ranks(values, dist, device):
    """Element-wise maximum of a list of floats over all ranks (the slowest rank sets the time)."""
    import torch
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(v) for v in values]
    t = torch.tensor(list(values), device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def whole_job_value(step_flops, world, ms_per_step):
    """Replicas only: every rank runs the same step on its own data, so the job does world x flops."""
    return world * step_flops / (ms_per_step * 1e-3) / 1e9


def run_ours(args):
    import torch
    import torch.distributed as dist

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)
    import paper_2211_10482_b200 as st
    st.lib()   # fails loudly when the CUDA library is missing

    peaks = load_peaks()
    cfg = bench_config()
    # the tensor-core variants are used when the library offers them for these shapes
    c5 = cfg["moment2_large"]
    if st.st_workspace_bytes(st.ST_OP_SYM_MOMENT2, c5["N"], c5["d"], st.ST_BF16) == 0 or args.m2_large == "f32":
        cfg["m2_large_dtype"] = "f32"
    if st.st_workspace_bytes(st.ST_OP_TTM_BLOCKDIAG, 64, 64, 256, 64, st.ST_FLAG_TC_TF32) == 0 or args.ttm == "f32":
        cfg["ttm_tc"] = False
    if args.mttkrp == "f32":
        cfg["mttkrp_tc"] = False
    w = Workload(cfg, device, st, torch)
    table = step_table(cfg)
    calls = w.calls()
    names = [n for n, _ in calls]
    torch.cuda.synchronize()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def one_step(events=None):
        for idx, (name, fn) in enumerate(calls):
            if events is not None:
                events[idx][0].record()
            fn()
            if events is not None:
                events[idx][1].record()

    for _ in range(args.warmup):
        one_step()
    barrier()
    if st.st_check_status(w.ws) != st.ST_OK:
        raise RuntimeError("a kernel reported a device-side error during warm-up")

    # ---- device-resident timing: K steps between two events; per-call events inside
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    ev = [[(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in calls]
          for _ in range(args.steps)]
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    t0.record()
    for s in range(args.steps):
        one_step(ev[s])
    t1.record()
    barrier()
    total_ms = t0.elapsed_time(t1)
    per_call_us = {n: float(np.mean([ev[s][i][0].elapsed_time(ev[s][i][1]) for s in range(args.steps)])) * 1e3
                   for i, n in enumerate(names)}

    # ---- end to end: host -> device copies of every input and device -> host of the results
    for _ in range(2):
        w.upload(); one_step(); w.download()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        w.upload()
        one_step()
        w.download()
    e1.record()
    barrier()
    e2e_ms = e0.elapsed_time(e1)
    clocks = sampler.stop() if rank == 0 else None   # sampled over both timed regions

    total_ms, e2e_ms = max_over_ranks([total_ms, e2e_ms], dist, device)

    step_flops = sum(table[n]["flops"] for n in names)
    ms_per_step = total_ms / args.steps
    value = whole_job_value(step_flops, world, ms_per_step)
    e2e_value = whole_job_value(step_flops, world, e2e_ms / args.steps)

    kernels = {}
    for n in names:
        us = per_call_us[n]
        rl = roofline_us(table[n], peaks)
        kernels[n] = {"us": round(us, 2), "gflops": round(table[n]["flops"] / us / 1e3, 1),
                      "gbs": round(table[n]["bytes"] / us / 1e3, 1), "roofline_us": round(rl, 2),
                      "frac": round(rl / us, 4), "bound": table[n]["bound"]}
    dominant = max(names, key=lambda n: per_call_us[n])
    dent, dus = table[dominant], per_call_us[dominant]
    if dent["bound"] == "hbm":
        roof = {"bound": "hbm", "achieved": dent["bytes"] / dus / 1e3, "peak": peaks["hbm_gbs"], "unit": "GB/s"}
    elif dent["bound"] == "tensor":
        roof = {"bound": "tensor", "achieved": dent["flops"] / dus / 1e6,
                "peak": peaks["bf16_tflops_sustained"] * dent.get("tensor_scale", 1.0), "unit": "TFLOP/s"}
    else:
        roof = {"bound": "alu", "achieved": dent["flops"] / dus / 1e6, "peak": FP32_PEAK_TFLOPS, "unit": "TFLOP/s"}
    roof["frac"] = roof["achieved"] / roof["peak"]
    tc_paths = {"sym_moment2_large": cfg["m2_large_dtype"] == "bf16", "ttm_blockdiag": cfg["ttm_tc"],
                "mttkrp_tri": cfg["mttkrp_tc"]}
    roof["traffic"] = NCU_TRAFFIC_BYTES.get(dominant) if tc_paths.get(dominant, False) else None
    roof["kernel"] = dominant
    roof["peak_source"] = ("derived from unit counts and clocks" if dent["bound"] == "alu" else
                           peaks["source"] + (" (sustained)" if dent["bound"] == "tensor" else ""))

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32" + ("+bf16" if cfg["m2_large_dtype"] == "bf16" else "") + ("+tf32" if (cfg["ttm_tc"] or cfg["mttkrp_tc"]) else ""),
        "data": "synthetic",
        "config": {"workload": "all five named configurations in one step: sym_moment2 [4096,64], sym_moment3 "
                               "[65536,64] (fp32, and its TF32 and bf16 tensor-core variants), sym_moment4 [65536,32] bf16, "
                               "thp on the packed mttkrp operand, mttkrp_tri I=K=512 R=32 (%s), ttm_blockdiag 64x(64x64) K=256 R=64 (%s), "
                               "sym_moment2 large [1048576,1024] %s; plus pack/unpack of their operands"
                               % ("tf32" if cfg["mttkrp_tc"] else "f32", "tf32" if cfg["ttm_tc"] else "f32",
                                  cfg["m2_large_dtype"]),
                   "l2": "inputs larger than L2 (each step streams >2.5 GB between two uses of any buffer)",
                   "replicas": "independent replicas, no collective" if world > 1 else "single GPU"},
        "roofline": roof,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": w.h2d_bytes, "d2h_bytes_per_step": w.d2h_bytes,
                "ms_per_step": e2e_ms / args.steps},
        "gpu_launches": args.steps * sum(table[n]["launches"] for n in names),
        "kernels": kernels, "clocks": clocks,
        "peaks": {"hbm_gbs": peaks["hbm_gbs"], "bf16_tflops": peaks.get("bf16_tflops"),
                  "bf16_tflops_sustained": peaks.get("bf16_tflops_sustained"), "fp32_tflops": FP32_PEAK_TFLOPS,
                  "source": peaks["source"]},
    }
    if world == 1 and not args.no_controls:
        line["dense_control"] = dense_controls(w, torch)
        line["sym_moment2_sample_sweep"] = moment2_sample_sweep(w, torch)
    if rank == 0:
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline(budget_s=args.cpu_budget)
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


# --------------------------------------------------------------------------------------
# the CPU oracle, timed as it stands on a bounded sample of the same step
# --------------------------------------------------------------------------------------

def oracle_sample_pass(sample):
    """One pass of the oracle over the sample; returns the useful flops of the sample."""
    import oracle
    flops = 0
    X1 = sample["X1"]
    oracle.moment2(X1)
    flops += 2 * X1.shape[0] * tri(X1.shape[1])
    X2 = sample["X2"]
    oracle.moment3(X2)
    flops += 2 * X2.shape[0] * tet(X2.shape[1]) + X2.shape[0] * tri(X2.shape[1])
    Bd, C, D, rows = sample["B3"], sample["C3"], sample["D3"], sample["rows3"]
    oracle.mttkrp(Bd, C, D, rows[0], rows[1])
    I, K, R = Bd.shape[0], Bd.shape[2], C.shape[1]
    uniq = sum(I - i for i in range(rows[0], rows[1]))
    flops += 2 * R * uniq * K + 2 * R * uniq
    B4, U4 = sample["B4"], sample["U4"]
    oracle.ttm(B4, U4)
    flops += 2 * B4.shape[0] * B4.shape[1] * U4.shape[1]
    X5 = sample["X5"]
    oracle.moment2(X5)
    flops += 2 * X5.shape[0] * tri(X5.shape[1])
    return flops


def make_sample():
    import oracle
    c = workloads.CONFIGS
    s = {}
    s["X1"] = workloads.moment_input("moment2")                      # whole configuration
    s["X2"] = workloads.moment_input("moment3", N=512)               # first 512 of 65536 samples
    I, K, R = 128, c["mttkrp"]["K"], c["mttkrp"]["R"]
    Bp, C, D = workloads.mttkrp_inputs(I, K, R)                      # I=128 instead of 512, 16 rows of A
    s["B3"] = oracle.unpack(Bp.reshape(-1), oracle.KIND_TRI, I, inner=K)
    s["C3"], s["D3"], s["rows3"] = C, D, (0, 16)
    Bp4, U4 = workloads.ttm_inputs(nb=1, bs=64)                      # one of the 64 blocks
    s["B4"], s["U4"] = Bp4.reshape(-1, c["ttm"]["K"]), U4
    bits = workloads.draw_rows_bf16(1024, c["moment2_large"]["d"], "normal", workloads.SEEDS["moment2_large"])
    s["X5"] = workloads.bf16_bits_to_f32(bits).reshape(1024, -1)     # first 1024 of 1048576 samples
    desc = ("sym_moment2 whole; sym_moment3 first 512 of 65536 samples; mttkrp I=128 (of 512), 16 rows of A; "
            "ttm 1 of 64 blocks; sym_moment2 large first 1024 of 1048576 samples; dense iteration space, fp64")
    return s, desc


def cpu_baseline(budget_s=20.0):
    import oracle
    oracle.build()
    sample, desc = make_sample()
    oracle_sample_pass(sample)   # page in
    n, t0, flops = 0, time.perf_counter(), 0
    while True:
        flops += oracle_sample_pass(sample)
        n += 1
        if time.perf_counter() - t0 > budget_s or n >= 100:
            break
    dt = time.perf_counter() - t0
    return {"value": flops / dt / 1e9, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": desc + "; %d passes in %.1f s" % (n, dt)}


def run_reference(args):
    if int(os.environ.get("RANK", "0")) != 0:
        return
    import oracle
    oracle.build()
    sample, desc = make_sample()
    for _ in range(max(1, min(args.warmup, 3))):
        oracle_sample_pass(sample)
    steps = min(args.steps, 20)
    t0, flops = time.perf_counter(), 0
    for _ in range(steps):
        flops += oracle_sample_pass(sample)
    dt = time.perf_counter() - t0
    value = flops / dt / 1e9
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT,
        "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": steps, "warmup": args.warmup,
        "ms_per_step": dt / steps * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": {"workload": "CPU oracle on a bounded sample of the five named configurations", "sample": desc},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-controls", action="store_true", help="skip the dense-iteration controls")
    ap.add_argument("--cpu-budget", type=float, default=15.0)
    ap.add_argument("--m2-large", default="bf16", choices=["bf16", "f32"])
    ap.add_argument("--ttm", default="tf32", choices=["tf32", "f32"])
    ap.add_argument("--mttkrp", default="tf32", choices=["tf32", "f32"])
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
