"""Host-side arithmetic of bench.py: the per-kernel roofline fractions from a per-kernel time table
and the algorithmic work of a step (no GPU needed)."""

import os
import sys

import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench  # noqa: E402
import workloads as WL  # noqa: E402


def test_solve_flop_counts_the_smaller_system_per_row_and_block():
    cfg = WL.CONFIGS["tiny"]  # B = 64
    M = torch.zeros((2, 128), dtype=torch.uint8)
    M[0, :10] = 1          # block 0 of row 0: s = 10 -> n = 10
    M[1, 64:64 + 60] = 1   # block 1 of row 1: s = 60 -> n = 4 (complement form)
    want = 0.0
    for s in (10, 0, 0, 60):
        n = min(s, 64 - s)
        want += n ** 3 / 3.0 + 2.0 * n * n + 2.0 * s * (64 - s)
    assert abs(bench.solve_flop([M], cfg) - want) < 1e-9


def test_roofline_by_kernel_from_a_time_table():
    cfg = WL.CONFIGS["tiny"]  # one 256 x 256 layer, B = 64, unstructured
    peaks = {"hbm_gbs": 1000.0, "bf16_tflops": 100.0, "bf16_tflops_sustained": 80.0}
    tr_f = {"thanos::(anonymous namespace)::tc_gemm_kernel(...)": [3, 2.0]}
    tr_s = {"void thanos::(anonymous namespace)::select_pass_kernel<2>(...)": [20, 0.75],
            "void thanos::(anonymous namespace)::select_rest_kernel<2>(...)": [4, 0.25],
            "thanos::(anonymous namespace)::tc_gemm_kernel(...)": [3, 0.5],
            "thanos::(anonymous namespace)::solve_rows_tile_kernel(...)": [4, 0.25]}
    M = torch.zeros((256, 256), dtype=torch.uint8)
    M[:, ::2] = 1
    out = bench.roofline_by_kernel(tr_f, tr_s, cfg, peaks, 50.0, [M], {256: 1})
    resid = sum(256.0 * (256 - j1) for j1 in range(0, 256, 64))
    upd = sum(256.0 * (256 - min(256, j1 + 64)) for j1 in range(0, 256, 64))
    sel = out["select_pass_kernel"]
    assert abs(sel["achieved"] - 4.0 * resid / 1e-3 / 1e9) < 0.1 and sel["bound"] == "hbm"
    assert abs(sel["frac"] - sel["achieved"] / 1000.0) < 1e-3
    upd_e = out["tc_gemm_kernel (sweep update)"]
    assert abs(upd_e["achieved"] - 8.0 * upd / 0.5e-3 / 1e9) < 0.1
    fac = out["tc_gemm_kernel (factorisation)"]
    assert abs(fac["achieved"] - (2.0 / 3.0) * 256.0 ** 3 / 2e-3 / 1e12) < 0.01 and fac["peak"] == 80.0
    sol = out["solve_rows kernels"]
    assert sol["bound"] == "alu" and sol["peak"] == 50.0
    assert abs(sol["achieved"] - bench.solve_flop([M], cfg) / 0.25e-3 / 1e12) < 0.01


def test_mode_selection_of_a_configuration():
    cfg = WL.CONFIGS["llama2_70b"]
    assert bench.select_mode(cfg, 0) is cfg
    alt = bench.select_mode(cfg, 1)
    assert alt.mode == "unstructured" and abs(alt.p - 0.6) < 1e-12 and alt.layers == cfg.layers
    assert bench.short_kernel_name("void thanos::(anonymous namespace)::foo_kernel<2>(int)") == "foo_kernel<2>"


def test_update_bytes_of_a_grouped_nm_sweep():
    """n:m sweeps of layers at least 2048 wide update in groups of 512 columns: the bytes an update
    changes are counted per group to the right of it, and the product is also rated as tensor work."""
    cfg = WL.CONFIGS["llama2_70b"]   # 2:4, B = 128: groups of four blocks
    assert cfg.mode == "nm" and cfg.B == 128
    peaks = {"hbm_gbs": 1000.0, "bf16_tflops": 100.0, "bf16_tflops_sustained": 80.0}
    tr_s = {"thanos::(anonymous namespace)::tc_gemm_pair_kernel(...)": [5, 1.0],
            "thanos::(anonymous namespace)::tc_gemm_kernel(...)": [5, 1.0]}
    out = bench.roofline_by_kernel({}, tr_s, cfg, peaks, 50.0, [], {})
    want = 0.0
    for L in cfg.layers:
        for j1 in range(0, L.b, 128):
            j2 = min(L.b, j1 + 128)
            ge = min(L.b, (j1 // 512 + 1) * 512)
            want += L.c * (ge - j2) + (L.c * (L.b - ge) if j2 == ge else 0)
    e = out["tc_gemm_kernel (sweep update)"]
    assert e["launches"] == 10 and abs(e["ms_per_step"] - 2.0) < 1e-9   # both kernels counted
    assert abs(e["achieved"] - 8.0 * want / 2e-3 / 1e9) / e["achieved"] < 1e-3
    flop = sum(float(L.c) * L.b * L.b for L in cfg.layers)
    assert abs(e["tensor_useful_tflops"] - flop / 2e-3 / 1e12) / e["tensor_useful_tflops"] < 1e-3
    assert abs(e["tensor_frac_executed"] - 6.0 * e["tensor_frac_useful"]) < 1e-3
