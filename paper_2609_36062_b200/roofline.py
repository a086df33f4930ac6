"""Algorithmic work of the chunkwise SMat prefill and the roofline it implies.

Counts are what the method itself has to do (Theorem 2's cost terms), per (batch, head), with
r = d_k, p = d_v, e = bytes per input element, fp32 tables:

  tensor flop (forward)  = T (c+1)(r+p)             within-chunk tril tiles (two products)
                         + 2rp (T + T + n + m)      chunk summaries, carried-state read, pool, typed read
  ALU adds   (forward)   = nnz(C) rp + (T/c) rp     Algorithm 2's state additions + the scan
  HBM bytes  (forward)   = (2r + 2p) T e            Q, K, V in, O out
                         + 2 P rp s_F + 2 B rp s_U  profile table and type table, written once and read once
                           (d = 1 has neither table; s = 4, or 2 where the implementation stores the table as
                           bf16 — the fraction against fp32 tables is reported beside the design's own)
  backward               = T (c+1)(3r+2p) + 15 T rp flop, the same adds again (Cᵀ tabulation, suffix scan),
                           (4r + 3p) T e bytes of tensors and 2 (2P + 2B) rp 4 bytes of tables
                           (F, U rebuilt; Ū, F̄ written and read)

Chunk-state traffic (T/c states written and read) depends on the implementation and is not counted.
Peaks come from MEASURED_PEAKS.json when present (HBM copy GB/s, dense bf16 TFLOP/s, both measured on
this machine's B200s), else from the stated fallback.  The fp32 add peak is the rate the library's add
microbenchmark measures on the device (bench.py puts it into the peaks), else nominal:
148 SMs x 128 lanes x the maximum SM clock.
"""
from __future__ import annotations

import json
import os
from dataclasses import dataclass

FALLBACK = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "sm_max_mhz": 1965.0}


def load_peaks(root: str) -> dict:
    path = os.path.join(root, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            data = json.load(f)
        data["source"] = "measured"
        return data
    data = dict(FALLBACK)
    data["source"] = "fallback"
    return data


@dataclass
class Work:
    flops: float       # dense contraction flop
    adds: float        # fp32 state additions on the plain ALUs
    bytes: float       # HBM bytes

    def __add__(self, o):
        return Work(self.flops + o.flops, self.adds + o.adds, self.bytes + o.bytes)

    def scaled(self, k):
        return Work(self.flops * k, self.adds * k, self.bytes * k)


def forward_work(T, c, r, p, e, geo, u_bytes=4, f_bytes=4) -> Work:
    """u_bytes, f_bytes: element sizes of the type and profile tables as the implementation keeps them (4, or 2
    where a table is stored as bf16)."""
    rp = r * p
    lr = geo.d > 1
    flops = T * (c + 1) * (r + p) + 2 * rp * (2 * T + (geo.n + geo.m if lr else 0))
    adds = (geo.nnzC * rp if lr else 0) + (T // c) * rp
    by = (2 * r + 2 * p) * T * e + (2 * geo.P * rp * f_bytes + 2 * geo.B * rp * u_bytes if lr else 0)
    return Work(flops, adds, by)


def backward_work(T, c, r, p, e, geo, u_bytes=4, fbar_bytes=4, keep_forward_tables=False, f_bytes=4,
                  ubar_bytes=4) -> Work:
    """Tables of the backward pass: Ū (fp32) and F̄ written and read once each, U read once; F and U rebuilt
    first (F written and read, U written) unless the forward's tables are kept in the workspace."""
    rp = r * p
    lr = geo.d > 1
    rebuilt = 0 if keep_forward_tables else 2
    flops = T * (c + 1) * (3 * r + 2 * p) + ((15 - (0 if rebuilt else 3)) if lr else 10) * T * rp
    adds = (geo.nnzC * rp * (2 if rebuilt else 1) if lr else 0) + 2 * (T // c) * rp
    tables = (rebuilt * geo.P * f_bytes + (rebuilt // 2) * geo.B * u_bytes   # F written + read, U written
              + geo.B * u_bytes                                        # U read by the dQ typed read
              + 2 * geo.B * ubar_bytes + 2 * geo.P * fbar_bytes) * rp  # Ū, F̄ written and read
    by = (4 * r + 3 * p) * T * e + (tables if lr else 0)
    return Work(flops, adds, by)


def roofline_times(work: Work, peaks: dict, sustained: bool = True) -> dict:
    """Seconds each ceiling needs for `work`, and the two path rooflines (2-term: every operation charged
    at the tensor peak against the HBM term; 3-term: table additions charged at the fp32 add peak)."""
    tflops = peaks["bf16_tflops_sustained" if sustained else "bf16_tflops"] * 1e12
    hbm = peaks["hbm_gbs"] * 1e9
    # fp32 add peak: measured on the device when the caller put it into `peaks` (bench.py does), else nominal
    alu = peaks.get("fadd_adds_per_s") or 148 * 128 * peaks.get("sm_max_mhz", 1965.0) * 1e6
    t_tensor = work.flops / tflops
    t_alu = work.adds / alu
    t_hbm = work.bytes / hbm
    t2 = max((work.flops + work.adds) / tflops, t_hbm)
    t3 = max(t_tensor, t_alu, t_hbm)
    return {"t_tensor": t_tensor, "t_alu": t_alu, "t_hbm": t_hbm, "t_2term": t2, "t_3term": t3, "alu_peak_adds": alu,
            "alu_peak_source": "measured" if peaks.get("fadd_adds_per_s") else "nominal"}


# Per-kernel algorithmic traffic (bytes), adds and flop, keyed by the stage names the library reports.
def stage_work(name: str, T, c, r, p, e, geo, u_bytes=4, f_bytes=4) -> Work:
    """What one forward stage has to do at the least: its contraction flop, Algorithm 2's additions where it
    tabulates, and the bytes of its inputs and outputs (scratch the stage exchanges with itself is not counted)."""
    rp, NC = r * p, T // c
    n, m, P, B = geo.n, geo.m, geo.P, geo.B
    st = 4 * rp
    su = u_bytes * rp
    sf = f_bytes * rp
    tc_tiles = T // 128
    table = {
        "pool":        Work(2 * n * rp, 0, n * (r + p) * e + P * st),
        "pool_tc":     Work(2 * n * rp, 0, n * (r + p) * e + P * sf),
        "tabulate":    Work(0, geo.nnzC * rp, P * st + B * su),
        "tabulate_tc": Work(0, geo.nnzC * rp, P * sf + B * su),
        "tabulate_regs": Work(0, geo.nnzC * rp, P * sf + B * su),      # the same sums on the fp32 ALUs (bf16 tables)
        "tabulate_bf16": Work(0, geo.nnzC * rp, P * sf + B * su),
        "bwd_tabulate_t_tc": Work(0, geo.nnzC * rp, B * su + P * sf),
        "bwd_pool_type_tc": Work(2 * m * rp, 0, m * (r + p) * e + B * su),
        "bwd_dq_type_tc": Work(2 * m * rp, 0, m * p * e + B * su + m * r * 2),
        "bwd_dk_profile_tc": Work(2 * n * rp, 0, n * p * e + P * sf + n * r * 2),
        "bwd_dv_profile_tc": Work(2 * n * rp, 0, n * r * e + P * sf + n * p * 2),
        "bwd_dkdv_profile_tc": Work(4 * n * rp, 0, n * (r + p) * e + P * sf + n * (r + p) * 2),
        "bwd_suffix_scan_tc": Work(2 * T * rp, tc_tiles * rp, T * (r + p) * e + tc_tiles * rp * 2),
        # dQ, dK, dV of every 128-token tile: eight 128 x 128 x 128 products per tile; reads Q, K, V, dO, the two
        # per-tile states and the three long-range buffers (bf16), writes the three gradients
        "bwd_tiles_fused_tc": Work(tc_tiles * 8 * 2 * 128 * 128 * 128, 0,
                                   T * (2 * r + 2 * p) * e + T * (2 * r + p) * e + 2 * tc_tiles * rp * 2 +
                                   (m * r + n * r + n * p) * 2),
        "segment_state_tc": Work(2 * T * rp, 0, T * (r + p) * e),
        "segment_scan": Work(0, 0, 0),
        "segment_output_tc": Work(T * 129 * (r + p) + 4 * T * rp, 0, T * (2 * r + 2 * p) * e + m * p * 2),
        "chunk_state": Work(2 * T * rp, 0, T * (r + p) * e + NC * st),
        "scan":        Work(0, NC * rp, 2 * NC * st),
        "scores":      Work(T * (c + 1) * r, 0, 2 * T * r * e + T * c * 4),
        "read_chunk":  Work(2 * T * rp, 0, T * r * e + NC * st + T * p * 4),
        "read_type":   Work(2 * m * rp, 0, m * r * e + B * st + 2 * m * p * 4),
        "read_type_tc": Work(2 * m * rp, 0, m * r * e + B * su + m * p * 2),
        "chunk_scan_tc": Work(2 * T * rp, tc_tiles * rp, T * (r + p) * e + tc_tiles * rp * 2),
        "chunk_output_tc": Work(T * 129 * (r + p) + 2 * T * rp, 0, T * (2 * r + 2 * p) * e + tc_tiles * rp * 2 + m * p * 4),
        "output":      Work(T * (c + 1) * p, 0, T * c * 4 + T * p * e + T * p * 4 + T * p * e),
    }
    aliases = {"gated_chunk_scan_tc": "chunk_scan_tc", "gated_chunk_output_tc": "chunk_output_tc",
               "bwd_gated_suffix_scan_tc": "bwd_suffix_scan_tc", "bwd_gated_tiles_fused_tc": "bwd_tiles_fused_tc"}
    return table.get(aliases.get(name, name), Work(0, 0, 0))


# Stages whose additions run on the fp32 ALUs (the other tabulations form the same sums on the tensor cores).
ALU_STAGES = ("tabulate", "tabulate_regs", "tabulate_bf16", "bwd_tabulate_t")
