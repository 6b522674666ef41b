#!/usr/bin/env python
"""Benchmark of the structured-tensor hot path.

One step = one pass of the hot path over the five named synthetic workloads, operands resident
in HBM: the large second moment (bf16 tensor cores), the third moment, MTTKRP on an
upper-half-cube tensor, TTM on a block-diagonal tensor, the small second moment, and the pack /
unpack calls that feed and reconstruct them.  Every call is also timed on its own with the L2
flushed before each repetition (median and minimum of 20), together with the other variants
of the calls (fp32 / TF32 side by side, tensor-core third moment, fourth moment, THP); the
fractions of the roofline are computed from those isolated times.

Metric: structured GFLOP/s = useful flops over the unique / non-zero iteration space per
second (one FMA = 2 flops, loop-invariant products counted once), and per call the achieved
fraction of its roofline.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
"""
from __future__ import annotations

import argparse
import hashlib
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
TF32_OVER_BF16 = 0.5     # nominal ratio of the dense TF32 and bf16 tensor rates


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


def ncu_traffic():
    """DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) of the kernels that were
    captured with ncu, from profiles/dram_traffic.json.  Every entry names the source file of its
    kernel and that file's hash at capture time: once the file has changed the entry reads as null."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.json")
    out = {}
    if not os.path.exists(path):
        return out
    with open(path) as f:
        table = json.load(f)
    for call, ent in table.items():
        src = os.path.join(ROOT, ent["source"])
        sha = hashlib.sha256(open(src, "rb").read()).hexdigest()[:16] if os.path.exists(src) else None
        out[call] = ent["bytes_per_launch"] if sha == ent.get("sha256_16") else None
    return out


def tri(d):
    return d * (d + 1) // 2


def tet(d):
    return d * (d + 1) * (d + 2) // 6


def simp4(d):
    return d * (d + 1) * (d + 2) * (d + 3) // 24


# --------------------------------------------------------------------------------------
# sizes, useful flops and algorithmic bytes of every call
# --------------------------------------------------------------------------------------

def call_table(cfg):
    """name -> dict(flops, bytes, bound, launches).  Bytes are algorithmic: packed operands read
    once plus outputs written once.  bound: what the roofline time of the call is made of --
    "alu" (fp32 FMA peak), "tensor" (bf16 tensor peak x tensor_scale) or "hbm"; the roofline time
    is always the slower of that and bytes / HBM bandwidth."""
    c1, c2, c3, c4, c5 = (cfg[k] for k in ("moment2", "moment3", "mttkrp", "ttm", "moment2_large"))
    t = {}
    t["sym_moment2"] = dict(flops=2 * c1["N"] * tri(c1["d"]), bytes=4 * (c1["N"] * c1["d"] + tri(c1["d"])),
                            bound="alu", launches=2)
    t["unpack_tri_sym"] = dict(flops=0, bytes=4 * (tri(c1["d"]) + c1["d"] ** 2), bound="hbm", launches=1)
    m3 = dict(flops=2 * c2["N"] * tet(c2["d"]) + c2["N"] * tri(c2["d"]), bytes=4 * (c2["N"] * c2["d"] + tet(c2["d"])))
    t["sym_moment3"] = dict(m3, bound="alu", launches=2)
    t["sym_moment3_tf32"] = dict(m3, bound="tensor", launches=2, tensor_scale=TF32_OVER_BF16)
    t["sym_moment3_bf16"] = dict(m3, bound="tensor", launches=2, tensor_scale=1.0)
    dw = cfg["moment3_wide_d"]         # the third moment beyond the 64 features of the named configuration
    t["sym_moment3_d%d" % dw] = dict(flops=2 * c2["N"] * tet(dw) + c2["N"] * tri(dw), bytes=4 * (c2["N"] * dw + tet(dw)),
                                     bound="alu", launches=2)
    for d4 in cfg["moment4_d"]:
        m4 = dict(flops=2 * c2["N"] * simp4(d4) + c2["N"] * tri(d4), bytes=4 * (c2["N"] * d4 + simp4(d4)))
        t["sym_moment4_d%d" % d4] = dict(m4, bound="tensor", launches=4, tensor_scale=1.0 / 3.0)   # split pair features, three products
        t["sym_moment4_d%d_bf16" % d4] = dict(m4, bound="tensor", launches=4, tensor_scale=1.0)
    t["unpack_tet_sym"] = dict(flops=0, bytes=4 * (tet(c2["d"]) + c2["d"] ** 3), bound="hbm", launches=1)
    nnz3 = tri(c3["I"]) * c3["K"]
    t["pack_tri_x_k"] = dict(flops=0, bytes=2 * 4 * nnz3, bound="hbm", launches=1)
    # THP of the packed upper-half-cube tensor with a dense one: packed operand, gathered dense operand, packed result
    t["thp_tri_x_k"] = dict(flops=nnz3, bytes=3 * 4 * nnz3, bound="hbm", launches=1)
    mk = dict(flops=2 * c3["R"] * nnz3 + 2 * c3["R"] * tri(c3["I"]), bytes=4 * (nnz3 + (2 * c3["I"] + c3["K"]) * c3["R"]))
    t["mttkrp_tri"] = dict(mk, bound="alu", launches=2)
    t["mttkrp_tri_tf32"] = dict(mk, bound="tensor", launches=2, tensor_scale=TF32_OVER_BF16)
    t["mttkrp_tri_split"] = dict(mk, bound="tensor", launches=2, tensor_scale=1.0 / 3.0)   # three bf16 products per term
    rows4 = c4["nb"] * c4["bs"] ** 2
    tt = dict(flops=2 * rows4 * c4["K"] * c4["R"], bytes=4 * (rows4 * (c4["K"] + c4["R"]) + c4["K"] * c4["R"]))
    t["ttm_blockdiag"] = dict(tt, bound="alu", launches=1)
    t["ttm_blockdiag_tf32"] = dict(tt, bound="tensor", launches=1, tensor_scale=TF32_OVER_BF16)
    t["ttm_blockdiag_split"] = dict(tt, bound="tensor", launches=1, tensor_scale=1.0 / 3.0)
    d4 = c4["nb"] * c4["bs"]
    t["unpack_blockdiag"] = dict(flops=0, bytes=4 * c4["R"] * (rows4 + d4 * d4), bound="hbm", launches=1)
    nb_, kw = cfg["band"]["d"], cfg["band"]["kl"] + cfg["band"]["ku"] + 1
    t["pack_band"] = dict(flops=0, bytes=2 * 4 * nb_ * kw * cfg["band"]["inner"], bound="hbm", launches=1)
    m2l = dict(flops=2 * c5["N"] * tri(c5["d"]))
    t["sym_moment2_large"] = dict(m2l, bytes=2 * c5["N"] * c5["d"] + 4 * tri(c5["d"]), bound="tensor", launches=2,
                                  tensor_scale=1.0)
    t["sym_moment2_large_f32"] = dict(m2l, bytes=4 * c5["N"] * c5["d"] + 4 * tri(c5["d"]), bound="alu", launches=2)
    t["sym_moment2_large_f32_tf32"] = dict(m2l, bytes=4 * c5["N"] * c5["d"] + 4 * tri(c5["d"]), bound="tensor", launches=2,
                                           tensor_scale=TF32_OVER_BF16)
    # three bf16 partial products per term; the split pass reads X and writes as many bytes, the GEMM passes read them again
    t["sym_moment2_large_f32_split"] = dict(m2l, bytes=4 * c5["N"] * c5["d"] + 4 * tri(c5["d"]), bound="tensor", launches=3,
                                            tensor_scale=1.0 / 3.0)
    t["unpack_tri_sym_large"] = dict(flops=0, bytes=4 * (tri(c5["d"]) + c5["d"] ** 2), bound="hbm", launches=1)
    return t


def tensor_peak_tflops(entry, peaks, burst):
    """bf16 tensor peak for a call: the burst figure for a kernel timed on its own, the sustained
    one inside the long step; TF32 calls take the measured TF32 yardstick when there is one, else
    the bf16 figure times the nominal TF32 / bf16 ratio."""
    scale = entry.get("tensor_scale", 1.0)
    if scale == TF32_OVER_BF16 and burst and peaks.get("tf32_tflops_yardstick"):
        return peaks["tf32_tflops_yardstick"]
    return peaks["bf16_tflops" if burst else "bf16_tflops_sustained"] * scale


def roofline_us(entry, peaks, burst=True):
    """Roofline time of one call: the slower of useful flops at peak and algorithmic bytes over the
    measured HBM bandwidth."""
    hbm = entry["bytes"] / (peaks["hbm_gbs"] * 1e9)
    if entry["bound"] == "tensor":
        alu = entry["flops"] / (tensor_peak_tflops(entry, peaks, burst) * 1e12)
    elif entry["bound"] == "hbm":
        alu = 0.0
    else:
        alu = entry["flops"] / (FP32_PEAK_TFLOPS * 1e12)
    return max(hbm, alu) * 1e6, ("hbm" if hbm >= alu else entry["bound"])


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
    cfg["moment3_wide_d"] = 128
    cfg["moment4_d"] = (32, 64)       # the fourth moment runs on the first d features of the third moment's samples
    return cfg


# The calls of one step (the hot path, one variant per call) in issue order.  Between the write of
# any buffer of 2 MB or more and its next read at least 400 MB stream through the 126 MB L2; only
# the two small reconstructions of the moment outputs read what the call before them left in L2.
STEP_CALLS = ["sym_moment2_large", "pack_tri_x_k", "unpack_tri_sym_large", "ttm_blockdiag_tf32", "pack_band",
              "unpack_blockdiag", "mttkrp_tri_split", "sym_moment3", "sym_moment2", "unpack_tet_sym", "unpack_tri_sym"]
# Timed on their own only (variants and widened rows)
EXTRA_CALLS = ["mttkrp_tri", "mttkrp_tri_tf32", "ttm_blockdiag", "ttm_blockdiag_split", "sym_moment3_tf32", "sym_moment3_bf16", "sym_moment3_d128", "sym_moment4_d32",
               "sym_moment4_d32_bf16", "sym_moment4_d64", "sym_moment4_d64_bf16", "thp_tri_x_k", "sym_moment2_large_f32",
               "sym_moment2_large_f32_tf32", "sym_moment2_large_f32_split"]


class Workload:
    """Host (pinned) and device copies of every input of one step, and the calls themselves."""

    def __init__(self, cfg, device, st, torch, extras=True):
        self.cfg, self.st, self.torch, self.device = cfg, st, torch, device
        c1, c2, c3, c4, c5 = (cfg[k] for k in ("moment2", "moment3", "mttkrp", "ttm", "moment2_large"))
        pin = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory()
        host = {}
        host["X1"] = pin(workloads.moment_input("moment2"))
        host["X2"] = pin(workloads.moment_input("moment3"))
        Bp3, C3, D3 = workloads.mttkrp_inputs()
        host["C3"], host["D3"] = pin(C3), pin(D3)
        Bp4, U4 = workloads.ttm_inputs()
        host["Bp4"], host["U4"] = pin(Bp4.reshape(-1, c4["K"])), pin(U4)
        bits = workloads.draw_rows_bf16(c5["N"], c5["d"], c5["dist"], workloads.SEEDS["moment2_large"])
        host["X5"] = torch.from_numpy(bits.view(np.int16)).pin_memory().view(torch.bfloat16)
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
            "m3": torch.empty(tet(c2["d"]), **f32), "m3_dense": torch.empty(c2["d"] ** 3, **f32),
            "Bp3": torch.empty(tri(c3["I"]) * c3["K"], **f32), "A3": torch.empty((c3["I"], c3["R"]), **f32),
            "Ap4": torch.empty((c4["nb"] * c4["bs"] ** 2, c4["R"]), **f32),
            "A4_dense": torch.empty((c4["nb"] * c4["bs"]) ** 2 * c4["R"], **f32),
            "band_p": torch.empty(st.st_packed_elems(self.lay_band), **f32),
            "m2l": torch.empty(tri(c5["d"]), **f32), "m2l_dense": torch.empty(c5["d"] ** 2, **f32),
        }
        TF, BF, SP = st.ST_FLAG_TC_TF32, st.ST_FLAG_TC_BF16, st.ST_FLAG_TC_SPLIT
        sizes = [
            st.st_workspace_bytes(st.ST_OP_SYM_MOMENT2, c1["N"], c1["d"], st.ST_F32),
            st.st_workspace_bytes(st.ST_OP_SYM_MOMENT3, c2["N"], c2["d"]),
            st.st_workspace_bytes(st.ST_OP_MTTKRP_TRI, c3["I"], c3["K"], c3["R"], 0, SP),
            st.st_workspace_bytes(st.ST_OP_TTM_BLOCKDIAG, c4["nb"], c4["bs"], c4["K"], c4["R"], TF),
            st.st_workspace_bytes(st.ST_OP_SYM_MOMENT2, c5["N"], c5["d"], st.ST_BF16), 256]
        if extras:
            sizes += [st.st_workspace_bytes(st.ST_OP_SYM_MOMENT3, c2["N"], c2["d"], 0, 0, TF),
                      st.st_workspace_bytes(st.ST_OP_SYM_MOMENT3, c2["N"], c2["d"], 0, 0, BF),
                      st.st_workspace_bytes(st.ST_OP_MTTKRP_TRI, c3["I"], c3["K"], c3["R"], 0, TF),
                      st.st_workspace_bytes(st.ST_OP_MTTKRP_TRI, c3["I"], c3["K"], c3["R"], 0, 0),
                      st.st_workspace_bytes(st.ST_OP_TTM_BLOCKDIAG, c4["nb"], c4["bs"], c4["K"], c4["R"], 0),
                      st.st_workspace_bytes(st.ST_OP_TTM_BLOCKDIAG, c4["nb"], c4["bs"], c4["K"], c4["R"], SP),
                      st.st_workspace_bytes(st.ST_OP_SYM_MOMENT2, c5["N"], c5["d"], st.ST_F32),
                      st.st_workspace_bytes(st.ST_OP_SYM_MOMENT3, c2["N"], cfg["moment3_wide_d"])]
            for d4 in cfg["moment4_d"]:
                sizes += [st.st_workspace_bytes(st.ST_OP_SYM_MOMENT4, c2["N"], d4, 0, 0, 0),
                          st.st_workspace_bytes(st.ST_OP_SYM_MOMENT4, c2["N"], d4, 0, 0, BF)]
        if min(sizes) <= 0:
            raise RuntimeError("the library does not cover one of the benchmark's shapes: %r" % (sizes,))
        self.ws = torch.empty(max(sizes), dtype=torch.uint8, device=device)
        self.h2d_bytes = sum(v.numel() * v.element_size() for v in host.values())
        self.result_keys = ["m2", "m3", "A3", "Ap4", "m2l"]
        self.host_out = {k: torch.empty_like(self.out[k], device="cpu").pin_memory() for k in self.result_keys}
        self.d2h_bytes = sum(v.numel() * v.element_size() for v in self.host_out.values())
        self._extra = None

    def calls(self):
        """name -> callable for the calls of the step."""
        st, d, o, c = self.st, self.dev, self.out, self.cfg
        c4 = c["ttm"]
        ws = self.ws
        return {
            "sym_moment2_large": lambda: st.st_sym_moment2(d["X5"], out=o["m2l"], ws=ws),
            "pack_tri_x_k": lambda: st.st_pack(d["B3"], self.lay3, out=o["Bp3"]),
            "unpack_tri_sym_large": lambda: st.st_unpack(o["m2l"], self.lay5, st.ST_FILL_SYMMETRIC, out=o["m2l_dense"]),
            "ttm_blockdiag_tf32": lambda: st.st_ttm_blockdiag(d["Bp4"], d["U4"], c4["nb"], c4["bs"], out=o["Ap4"], ws=ws,
                                                              flags=st.ST_FLAG_TC_TF32),
            "pack_band": lambda: st.st_pack(d["band"], self.lay_band, out=o["band_p"]),
            "unpack_blockdiag": lambda: st.st_unpack(o["Ap4"].view(-1), self.lay4, out=o["A4_dense"]),
            "mttkrp_tri_split": lambda: st.st_mttkrp_tri(o["Bp3"], d["C3"], d["D3"], out=o["A3"], ws=ws,
                                                         flags=st.ST_FLAG_TC_SPLIT),
            "sym_moment3": lambda: st.st_sym_moment3(d["X2"], out=o["m3"], ws=ws),
            "sym_moment2": lambda: st.st_sym_moment2(d["X1"], out=o["m2"], ws=ws),
            "unpack_tet_sym": lambda: st.st_unpack(o["m3"], self.lay2, st.ST_FILL_SYMMETRIC, out=o["m3_dense"]),
            "unpack_tri_sym": lambda: st.st_unpack(o["m2"], self.lay1, st.ST_FILL_SYMMETRIC, out=o["m2_dense"]),
        }

    def extra_calls(self):
        """name -> callable for the variants and widened rows that are timed on their own."""
        st, d, o, c, torch = self.st, self.dev, self.out, self.cfg, self.torch
        c4 = c["ttm"]
        ws = self.ws
        f32 = dict(dtype=torch.float32, device=self.device)
        if self._extra is None:
            self._extra = {"thp3": torch.empty_like(o["Bp3"]), "m3_tc": torch.empty_like(o["m3"])}
            dw = c["moment3_wide_d"]
            gen = torch.Generator(device=self.device).manual_seed(workloads.SEEDS["moment3"] + dw)
            self._extra["X3w"] = torch.randn((c["moment3"]["N"], dw), generator=gen, **f32)
            self._extra["m3w"] = torch.empty(tet(dw), **f32)
            for d4 in c["moment4_d"]:
                self._extra["X4_%d" % d4] = d["X2"][:, :d4].contiguous()
                self._extra["m4_%d" % d4] = torch.empty(simp4(d4), **f32)
        x = self._extra
        calls = {
            "mttkrp_tri": lambda: st.st_mttkrp_tri(o["Bp3"], d["C3"], d["D3"], out=o["A3"], ws=ws),
            "ttm_blockdiag_split": lambda: st.st_ttm_blockdiag(d["Bp4"], d["U4"], c4["nb"], c4["bs"], out=o["Ap4"], ws=ws,
                                                               flags=st.ST_FLAG_TC_SPLIT),
            "mttkrp_tri_tf32": lambda: st.st_mttkrp_tri(o["Bp3"], d["C3"], d["D3"], out=o["A3"], ws=ws, flags=st.ST_FLAG_TC_TF32),
            "ttm_blockdiag": lambda: st.st_ttm_blockdiag(d["Bp4"], d["U4"], c4["nb"], c4["bs"], out=o["Ap4"], ws=ws),
            "sym_moment3_tf32": lambda: st.st_sym_moment3(d["X2"], out=x["m3_tc"], ws=ws, flags=st.ST_FLAG_TC_TF32),
            "sym_moment3_bf16": lambda: st.st_sym_moment3(d["X2"], out=x["m3_tc"], ws=ws, flags=st.ST_FLAG_TC_BF16),
            "thp_tri_x_k": lambda: st.st_thp(o["Bp3"], d["B3"], self.lay3, out=x["thp3"]),
            "sym_moment3_d%d" % c["moment3_wide_d"]: lambda: st.st_sym_moment3(x["X3w"], out=x["m3w"], ws=ws),
        }
        for d4 in c["moment4_d"]:
            calls["sym_moment4_d%d" % d4] = (lambda d4=d4: st.st_sym_moment4(x["X4_%d" % d4], out=x["m4_%d" % d4], ws=ws))
            calls["sym_moment4_d%d_bf16" % d4] = (lambda d4=d4: st.st_sym_moment4(x["X4_%d" % d4], out=x["m4_%d" % d4], ws=ws,
                                                                                  flags=st.ST_FLAG_TC_BF16))
        return calls

    def upload(self):
        for k, v in self.host.items():
            self.dev[k].copy_(v, non_blocking=True)

    def download(self):
        for k in self.result_keys:
            self.host_out[k].copy_(self.out[k], non_blocking=True)


class Isolated:
    """Times one call on its own: the L2 is flushed before every repetition, and the flush keeps the GPU
    busy while the host queues the call, so that the two events bracket GPU time only.  The flush
    overwrites a 256 MB buffer and then (clean=True) reads another 256 MB: after the write alone about
    100 MB of the flush buffer sit in the L2 as dirty lines, and their write-back to HBM would run inside
    the timed region, on top of the traffic of the call (10 us and more on the streaming calls)."""

    def __init__(self, torch, device):
        self.torch = torch
        self.flush = torch.empty(256 << 20, dtype=torch.uint8, device=device)
        self.sweep = torch.zeros(64 << 20, dtype=torch.float32, device=device)

    def __call__(self, fn, reps=20, warm=3, clean=True):
        torch = self.torch
        for _ in range(warm):
            fn()
        torch.cuda.synchronize()
        # all repetitions are queued before the one synchronisation, so that the GPU never idles (and never
        # leaves its boost clock) between a flush and the call it precedes
        pairs = []
        for _ in range(reps):
            self.flush.zero_()
            if clean:
                self.sweep.sum()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            fn()
            e1.record()
            pairs.append((e0, e1))
        torch.cuda.synchronize()
        ts = [e0.elapsed_time(e1) * 1e3 for e0, e1 in pairs]
        return float(np.median(ts)), float(min(ts))


def tf32_yardstick(torch, device):
    """Dense TF32 matmul rate of torch (cuBLAS) on this GPU: a yardstick for the TF32 tensor peak
    only -- no part of the library calls it."""
    n = 8192
    a = torch.randn(n, n, device=device)
    b = torch.randn(n, n, device=device)
    old = torch.backends.cuda.matmul.allow_tf32
    torch.backends.cuda.matmul.allow_tf32 = True
    try:
        for _ in range(3):
            torch.matmul(a, b)
        torch.cuda.synchronize()
        ts = []
        for _ in range(5):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            torch.matmul(a, b)
            e1.record()
            torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1))
    finally:
        torch.backends.cuda.matmul.allow_tf32 = old
    return 2.0 * n ** 3 / (min(ts) * 1e-3) / 1e12


def dense_controls(w, timer, torch):
    """Every compute kernel against the same kernel forced onto the dense, unstructured iteration
    space (ST_FLAG_DENSE_CONTROL): isolated timings with an L2 flush between repetitions.  The
    gain from structure should approach dense work / unique work."""
    st, d, o, c = w.st, w.dev, w.out, w.cfg
    c1, c2, c3, c4, c5 = (c[k] for k in ("moment2", "moment3", "mttkrp", "ttm", "moment2_large"))
    DC, TF, SP = st.ST_FLAG_DENSE_CONTROL, st.ST_FLAG_TC_TF32, st.ST_FLAG_TC_SPLIT
    dev = w.device
    wsb = max(st.st_workspace_bytes(st.ST_OP_SYM_MOMENT2, c1["N"], c1["d"], st.ST_F32, 0, DC),
              st.st_workspace_bytes(st.ST_OP_SYM_MOMENT3, c2["N"], c2["d"], 0, 0, DC),
              st.st_workspace_bytes(st.ST_OP_MTTKRP_TRI, c3["I"], c3["K"], c3["R"], 0, DC),
              st.st_workspace_bytes(st.ST_OP_MTTKRP_TRI, c3["I"], c3["K"], c3["R"], 0, DC | TF),
              st.st_workspace_bytes(st.ST_OP_MTTKRP_TRI, c3["I"], c3["K"], c3["R"], 0, DC | SP),
              st.st_workspace_bytes(st.ST_OP_SYM_MOMENT2, c5["N"], c5["d"], st.ST_BF16, 0, DC), 256)
    wsc = torch.empty(wsb, dtype=torch.uint8, device=dev)
    d4 = c4["nb"] * c4["bs"]
    lay4k = st.Layout(st.ST_BLOCKDIAG, d4, inner=c4["K"], nblocks=c4["nb"], bs=c4["bs"])
    B4_dense = st.st_unpack(d["Bp4"].view(-1), lay4k)                # 16 GiB: zeros off the diagonal blocks
    A4_dense = torch.empty((d4 * d4, c4["R"]), dtype=torch.float32, device=dev)
    pairs = {
        "sym_moment2": (lambda: st.st_sym_moment2(d["X1"], out=o["m2"], ws=w.ws),
                        lambda: st.st_sym_moment2(d["X1"], out=o["m2"], ws=wsc, flags=DC), c1["d"] ** 2 / tri(c1["d"]), 20),
        "sym_moment3": (lambda: st.st_sym_moment3(d["X2"], out=o["m3"], ws=w.ws),
                        lambda: st.st_sym_moment3(d["X2"], out=o["m3"], ws=wsc, flags=DC), c2["d"] ** 3 / tet(c2["d"]), 10),
        "mttkrp_tri": (lambda: st.st_mttkrp_tri(o["Bp3"], d["C3"], d["D3"], out=o["A3"], ws=w.ws),
                       lambda: st.st_mttkrp_tri(d["B3"], d["C3"], d["D3"], out=o["A3"], ws=wsc, flags=DC),
                       c3["I"] ** 2 / tri(c3["I"]), 10),
        "mttkrp_tri_tf32": (lambda: st.st_mttkrp_tri(o["Bp3"], d["C3"], d["D3"], out=o["A3"], ws=w.ws, flags=TF),
                            lambda: st.st_mttkrp_tri(d["B3"], d["C3"], d["D3"], out=o["A3"], ws=wsc, flags=DC | TF),
                            c3["I"] ** 2 / tri(c3["I"]), 10),
        "mttkrp_tri_split": (lambda: st.st_mttkrp_tri(o["Bp3"], d["C3"], d["D3"], out=o["A3"], ws=w.ws, flags=SP),
                             lambda: st.st_mttkrp_tri(d["B3"], d["C3"], d["D3"], out=o["A3"], ws=wsc, flags=DC | SP),
                             c3["I"] ** 2 / tri(c3["I"]), 10),
        "ttm_blockdiag": (lambda: st.st_ttm_blockdiag(d["Bp4"], d["U4"], c4["nb"], c4["bs"], out=o["Ap4"], ws=w.ws),
                          lambda: st.st_ttm_blockdiag(B4_dense, d["U4"], c4["nb"], c4["bs"], out=A4_dense, ws=w.ws, flags=DC),
                          float(c4["nb"]), 3),
        "ttm_blockdiag_tf32": (lambda: st.st_ttm_blockdiag(d["Bp4"], d["U4"], c4["nb"], c4["bs"], out=o["Ap4"], ws=w.ws, flags=TF),
                               lambda: st.st_ttm_blockdiag(B4_dense, d["U4"], c4["nb"], c4["bs"], out=A4_dense, ws=w.ws,
                                                           flags=DC | TF), float(c4["nb"]), 3),
        "sym_moment2_large": (lambda: st.st_sym_moment2(d["X5"], out=o["m2l"], ws=w.ws),
                              lambda: st.st_sym_moment2(d["X5"], out=o["m2l"], ws=wsc, flags=DC),
                              c5["d"] ** 2 / tri(c5["d"]), 5),
    }
    out = {}
    for name, (structured, control, ideal, reps) in pairs.items():
        (a, amin), (b, bmin) = timer(structured, reps=reps, warm=2), timer(control, reps=reps, warm=1)
        out[name] = {"structured_us": round(a, 2), "control_us": round(b, 2), "ratio": round(b / a, 3),
                     "dense_over_unique": round(ideal, 3)}
    del B4_dense, A4_dense
    return out


def moment2_sample_sweep(w, timer, torch, peaks):
    """The small second moment (d = 64) from the named size up to 4M samples: the named size is bound by
    launch and memory latency, the sweep shows where the kernel reaches its fp32 roofline."""
    st = w.st
    dev = w.device
    d = w.cfg["moment2"]["d"]
    out = torch.empty(tri(d), dtype=torch.float32, device=dev)
    res = []
    for N in (4096, 32768, 262144, 1048576, 4194304):
        X = torch.empty((N, d), dtype=torch.float32, device=dev).uniform_(-1.0, 1.0)
        ws = torch.empty(max(st.st_workspace_bytes(st.ST_OP_SYM_MOMENT2, N, d, st.ST_F32), 256), dtype=torch.uint8, device=dev)
        us, us_min = timer(lambda: st.st_sym_moment2(X, out=out, ws=ws), reps=10, warm=2)
        flops, nbytes = 2 * N * tri(d), 4 * (N * d + tri(d))
        roof = max(flops / (FP32_PEAK_TFLOPS * 1e12), nbytes / (peaks["hbm_gbs"] * 1e9)) * 1e6
        res.append({"N": N, "us": round(us, 2), "us_min": round(us_min, 2), "tflops": round(flops / us / 1e6, 2),
                    "gbs": round(nbytes / us / 1e3, 1), "roofline_us": round(roof, 2), "frac": round(roof / us, 4)})
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
    extras = world == 1 and not args.no_isolated
    w = Workload(cfg, device, st, torch, extras=extras)
    table = call_table(cfg)
    step_calls = w.calls()
    names = list(STEP_CALLS)
    fns = [step_calls[n] for n in names]
    torch.cuda.synchronize()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def one_step(events=None):
        for idx, fn in enumerate(fns):
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
    ev = [[(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in names]
          for _ in range(args.steps)]
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    t0.record()
    for s in range(args.steps):
        one_step(ev[s])
    t1.record()
    barrier()
    total_ms = t0.elapsed_time(t1)
    in_step = {n: [ev[s][i][0].elapsed_time(ev[s][i][1]) * 1e3 for s in range(args.steps)] for i, n in enumerate(names)}

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

    # ---- every call on its own, L2 flushed
    timer = Isolated(torch, device)
    isolated = {}
    dirty = {}          # the same with the write-only flush: dirty lines of the flush buffer left in the L2
    if extras:
        peaks["tf32_tflops_yardstick"] = round(tf32_yardstick(torch, device), 1)
        every = dict(step_calls)
        every.update(w.extra_calls())
        c5 = cfg["moment2_large"]
        X5f = None
        for n in names + EXTRA_CALLS:
            if n in ("sym_moment2_large_f32_tf32", "sym_moment2_large_f32_split"):
                continue                             # timed together with the fp32 FMA path below
            if n == "sym_moment2_large_f32":       # the fp32 copy of the large input lives only for these two measurements
                X5f = w.dev["X5"].float()
                m2f = torch.empty_like(w.out["m2l"])
                isolated[n] = timer(lambda: st.st_sym_moment2(X5f, out=m2f, ws=w.ws), reps=3, warm=1)
                for name, flag in (("sym_moment2_large_f32_tf32", st.ST_FLAG_TC_TF32), ("sym_moment2_large_f32_split", st.ST_FLAG_TC_SPLIT)):
                    wst = torch.empty(st.st_workspace_bytes(st.ST_OP_SYM_MOMENT2, X5f.shape[0], X5f.shape[1], st.ST_F32, 0, flag),
                                      dtype=torch.uint8, device=device)
                    tf = lambda: st.st_sym_moment2(X5f, out=m2f, ws=wst, flags=flag)
                    isolated[name] = timer(tf, reps=10, warm=2)
                    dirty[name] = timer(tf, reps=5, warm=1, clean=False)
                    if st.st_check_status(wst) != st.ST_OK:
                        raise RuntimeError("the tensor-core second moment on fp32 input reported a device-side error")
                    del wst
                del X5f, m2f
                continue
            big = table[n]["bytes"] > (1 << 30) or n.startswith("sym_moment2_large")
            isolated[n] = timer(every[n], reps=(10 if big else 20), warm=3)
            dirty[n] = timer(every[n], reps=(5 if big else 10), warm=1, clean=False)
        if st.st_check_status(w.ws) != st.ST_OK:
            raise RuntimeError("a kernel reported a device-side error during the isolated timings")

    kernels = {}
    for n in (names + EXTRA_CALLS if extras else names):
        ent = {"bound": table[n]["bound"], "flops": table[n]["flops"], "bytes": table[n]["bytes"]}
        if n in in_step:
            ent["in_step_us"] = round(float(np.median(in_step[n])), 2)
            ent["in_step_us_min"] = round(float(min(in_step[n])), 2)
        if n in isolated:
            us, us_min = isolated[n]
            rl, bound = roofline_us(table[n], peaks, burst=True)
            ent.update({"us": round(us, 2), "us_min": round(us_min, 2), "gflops": round(table[n]["flops"] / us / 1e3, 1),
                        "gbs": round(table[n]["bytes"] / us / 1e3, 1), "roofline_us": round(rl, 2), "roofline_of": bound,
                        "frac": round(rl / us, 4)})
            if n in dirty:
                ent["us_dirty_l2"] = round(dirty[n][0], 2)
        else:
            rl, bound = roofline_us(table[n], peaks, burst=False)
            us = ent["in_step_us"]
            ent.update({"roofline_us": round(rl, 2), "roofline_of": bound, "frac_in_step": round(rl / us, 4)})
        kernels[n] = ent

    # the roofline object: the call with the largest share of the step, on its isolated time when there is one
    dominant = max(names, key=lambda n: float(np.median(in_step[n])))
    dent = table[dominant]
    burst = dominant in isolated
    dus = isolated[dominant][0] if burst else float(np.median(in_step[dominant]))
    rl, bound = roofline_us(dent, peaks, burst=burst)
    if bound == "hbm":
        roof = {"bound": "hbm", "achieved": dent["bytes"] / dus / 1e3, "peak": peaks["hbm_gbs"], "unit": "GB/s"}
    elif bound == "tensor":
        roof = {"bound": "tensor", "achieved": dent["flops"] / dus / 1e6, "peak": tensor_peak_tflops(dent, peaks, burst),
                "unit": "TFLOP/s"}
    else:
        roof = {"bound": "alu", "achieved": dent["flops"] / dus / 1e6, "peak": FP32_PEAK_TFLOPS, "unit": "TFLOP/s"}
    roof["frac"] = roof["achieved"] / roof["peak"]
    roof["traffic"] = ncu_traffic().get(dominant)
    roof["kernel"] = dominant
    roof["timing"] = ("isolated launch, L2 flushed (256 MB written, then 256 MB read), median of %d" % 10) if burst else "inside the step"
    roof["peak_source"] = ("derived from unit counts and clocks" if bound == "alu" else
                           peaks["source"] + ((" (burst)" if burst else " (sustained)") if bound == "tensor" else ""))

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32+bf16+tf32", "data": "synthetic",
        "config": {"workload": "the five named configurations in one step, one variant each: sym_moment2 large [1048576,1024] bf16 "
                               "tensor cores; sym_moment3 [65536,64] fp32; mttkrp_tri I=K=512 R=32 split-bf16 tensor cores (fp32 tolerance); ttm_blockdiag "
                               "64x(64x64) K=256 R=64 TF32 tensor cores; sym_moment2 [4096,64] fp32; plus the pack / unpack "
                               "calls of their operands and results (tri x K, band, block-diagonal, symmetric fills)",
                   "step_calls": names,
                   "l2": "inputs larger than L2: between the write of any buffer of 2 MB or more and its next read at least "
                         "400 MB stream through the 126 MB L2; the two small symmetric reconstructions read the moment "
                         "outputs (<= 183 KB) that the call before them left in L2.  The per-call fractions come from "
                         "isolated launches with the L2 flushed before each repetition (kernels[*].us: 256 MB written, then "
                         "256 MB of another buffer read so that no dirty line of the flush is written back inside the timed "
                         "region; kernels[*].us_dirty_l2 is the same call after the write alone), not from the step",
                   "replicas": "independent replicas, no collective" if world > 1 else "single GPU"},
        "roofline": roof,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": w.h2d_bytes, "d2h_bytes_per_step": w.d2h_bytes,
                "ms_per_step": e2e_ms / args.steps},
        "gpu_launches": args.steps * sum(table[n]["launches"] for n in names),
        "kernels": kernels, "clocks": clocks,
        "peaks": {"hbm_gbs": peaks["hbm_gbs"], "bf16_tflops": peaks.get("bf16_tflops"),
                  "bf16_tflops_sustained": peaks.get("bf16_tflops_sustained"),
                  "tf32_tflops_yardstick": peaks.get("tf32_tflops_yardstick"), "fp32_tflops": FP32_PEAK_TFLOPS,
                  "source": peaks["source"],
                  "note": "isolated calls: bf16 burst peak, TF32 calls the torch TF32 matmul yardstick; fp32 derived from "
                          "unit counts and clocks"},
    }
    if extras and not args.no_controls:
        line["dense_control"] = dense_controls(w, timer, torch)
        line["sym_moment2_sample_sweep"] = moment2_sample_sweep(w, timer, torch, peaks)
    if rank == 0:
        if world == 1 and not args.no_cpu_baseline:
            del w
            line["cpu_baseline"] = cpu_baseline(budget_s=args.cpu_budget)
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


# --------------------------------------------------------------------------------------
# the CPU oracle, timed as it stands on bounded samples of the five configurations
# --------------------------------------------------------------------------------------

def oracle_samples(scale=1):
    """One bounded sample per named configuration: (name, description, extrapolated, useful flops of the
    sample, callable).  `scale` widens the samples that are cut along a linear dimension (used for the
    run on all cores).  The oracle iterates the FULL dense space of each sample in fp64."""
    import oracle
    c = workloads.CONFIGS
    out = []
    X1 = workloads.moment_input("moment2")
    out.append(("sym_moment2", "whole configuration [4096,64]", False, 2 * X1.shape[0] * tri(X1.shape[1]),
                lambda: oracle.moment2(X1)))
    n2 = min(c["moment3"]["N"], 4096 * scale)
    X2 = workloads.moment_input("moment3", N=n2)
    out.append(("sym_moment3", "first %d of %d samples (time is linear in the sample count)" % (n2, c["moment3"]["N"]),
                n2 < c["moment3"]["N"], 2 * n2 * tet(64) + n2 * tri(64), lambda: oracle.moment3(X2)))
    I, K, R = c["mttkrp"]["I"], c["mttkrp"]["K"], c["mttkrp"]["R"]
    Bp, C, D = workloads.mttkrp_inputs()
    Bd = oracle.unpack(Bp.reshape(-1), oracle.KIND_TRI, I, inner=K)
    del Bp
    r3 = min(I, 128 * scale)
    uniq = sum(I - i for i in range(r3))
    out.append(("mttkrp_tri", "rows 0..%d of the %d rows of A, full J x K range of the dense tensor" % (r3 - 1, I),
                r3 < I, 2 * R * uniq * K + 2 * R * uniq, lambda: oracle.mttkrp(Bd, C, D, 0, r3)))
    nb, bs, K4, R4 = (c["ttm"][k] for k in ("nb", "bs", "K", "R"))
    Bp4, U4 = workloads.ttm_inputs(nb=1, bs=bs)
    d4 = nb * bs
    r4 = min(d4, 16 * scale)
    # r4 rows i of the dense [d,d,K] tensor: bs fibres per row lie in the diagonal block, the others are zero
    Bdense = np.zeros((r4, d4, K4), np.float32)
    Bdense[:, :bs, :] = Bp4.reshape(bs, bs, K4)[:r4]
    out.append(("ttm_blockdiag", "%d of the %d rows i of the dense tensor (all %d fibres of each row, zero blocks included)"
                % (r4, d4, d4), True, 2 * r4 * bs * K4 * R4, lambda: oracle.ttm(Bdense.reshape(-1, K4), U4)))
    n5 = 1024 * scale
    bits = workloads.draw_rows_bf16(n5, c["moment2_large"]["d"], "normal", workloads.SEEDS["moment2_large"])
    X5 = workloads.bf16_bits_to_f32(bits).reshape(n5, -1)
    out.append(("sym_moment2_large", "first %d of %d samples (time is linear in the sample count)" % (n5, c["moment2_large"]["N"]),
                True, 2 * n5 * tri(1024), lambda: oracle.moment2(X5)))
    return out


def time_oracle(fn, min_s=0.4):
    fn()                                  # page in
    n, t0 = 0, time.perf_counter()
    while True:
        fn()
        n += 1
        dt = time.perf_counter() - t0
        if dt > min_s:
            return dt / n


def cpu_baseline(budget_s=20.0):
    """The oracle as it stands, one thread and all cores, one entry per configuration.  `value` pools
    the all-core runs (useful flops of the samples over their time)."""
    import oracle
    oracle.build()
    cores = len(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else (os.cpu_count() or 1)
    per, flops_all, t_all = [], 0.0, 0.0
    singles = oracle_samples(1)
    multis = oracle_samples(4 if cores >= 8 else 1)
    for (name, desc1, ex1, fl1, fn1), (_, descn, exn, fln, fnn) in zip(singles, multis):
        oracle.set_threads(1)
        t1 = time_oracle(fn1)
        oracle.set_threads(cores)
        tn = time_oracle(fnn)
        flops_all += fln
        t_all += tn
        per.append({"config": name, "one_thread": {"gflops": round(fl1 / t1 / 1e9, 3), "seconds": round(t1, 3),
                                                    "sample": desc1, "cut_from_full_size": ex1},
                    "all_cores": {"gflops": round(fln / tn / 1e9, 3), "seconds": round(tn, 3), "sample": descn,
                                  "cut_from_full_size": exn}})
    return {"value": flops_all / t_all / 1e9, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": "per configuration a bounded sample of the dense fp64 iteration (see per_config[*].sample); value pools "
                      "the all-core runs; useful (structured) flops of the sample over oracle time",
            "per_config": per}


def run_reference(args):
    if int(os.environ.get("RANK", "0")) != 0:
        return
    import oracle
    oracle.build()
    cores = len(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else (os.cpu_count() or 1)
    oracle.set_threads(cores)
    samples = oracle_samples(1)
    desc = "; ".join("%s: %s" % (n, d) for n, d, _, _, _ in samples)

    def one_pass():
        for _, _, _, _, fn in samples:
            fn()

    for _ in range(max(1, min(args.warmup, 3))):
        one_pass()
    steps = min(args.steps, 20)
    t0 = time.perf_counter()
    for _ in range(steps):
        one_pass()
    dt = time.perf_counter() - t0
    value = steps * sum(fl for _, _, _, fl, _ in samples) / dt / 1e9
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT,
        "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": steps, "warmup": args.warmup,
        "ms_per_step": dt / steps * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": {"workload": "CPU oracle on a bounded sample of each of the five named configurations", "sample": desc},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc},
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
    ap.add_argument("--no-controls", action="store_true", help="skip the dense-iteration controls and the sample sweep")
    ap.add_argument("--no-isolated", action="store_true", help="skip the per-call isolated timings (and what builds on them)")
    ap.add_argument("--cpu-budget", type=float, default=15.0)
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
