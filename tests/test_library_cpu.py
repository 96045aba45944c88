"""CPU-only checks of the C-ABI library: it loads, exports what the header declares, validates
arguments before touching a device, and its host-side placement matches the oracle."""
import ctypes as C
import os
import re

import numpy as np
import pytest
import torch

from oracle import c2r_oracle as O
from paper_2504_01337_b200 import inputs as G

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def b():
    from paper_2504_01337_b200 import build
    build.build()
    from paper_2504_01337_b200 import binding
    return binding


def test_exports_match_header(b):
    header = open(os.path.join(ROOT, "include", "c2r.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(c2r_[a-z0-9_]+)\s*\(", header))
    assert declared, "no declarations found"
    for name in declared:
        assert hasattr(b.lib, name), name
    assert declared == set(b.EXPORTS)


def test_struct_layout_matches_header(b):
    header = open(os.path.join(ROOT, "include", "c2r.h")).read()
    body = re.search(r"typedef struct c2r_layer_buffers \{(.*?)\} c2r_layer_buffers;", header, flags=re.S).group(1)
    body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
    names = re.findall(r"\b(\w+)\s*;", body)
    assert names == [n for n, _ in b.LayerBuffers._fields_]
    cbody = re.search(r"typedef struct c2r_config \{(.*?)\} c2r_config;", header, flags=re.S).group(1)
    cbody = re.sub(r"/\*.*?\*/", "", cbody, flags=re.S)
    assert re.findall(r"int32_t\s+(\w+)\s*;", cbody) == [n for n, _ in b.Config._fields_]


def test_sizes_and_argument_checks_need_no_gpu(b):
    cfg = b.make_config(16384, 2048, 60, 1408, 4, 16, 4, 5632, b.BF16, 128)
    assert b.permuted_rows(cfg) == 16384 * 4 + 60 * 127 + (128 - (16384 * 4 + 60 * 127) % 128) % 128
    assert b.workspace_bytes(cfg, b.WS_LAYER) >= b.workspace_bytes(cfg, b.WS_PERMUTE) > 0
    assert b.lib.c2r_route(C.byref(cfg), None, None, None, None, None, None, None, None) == -1
    bad = b.make_config(16, 60, 8, 16, 2, 1, 1, 0, b.BF16, 1)     # d % 8 != 0
    assert b.lib.c2r_gate_logits(C.byref(bad), None, None, None, None, None, None) == -2
    bad = b.make_config(16, 64, 65, 16, 2, 1, 1, 0, b.BF16, 1)    # E > 64
    assert b.lib.c2r_permuted_rows(C.byref(bad)) == -1
    bad = b.make_config(16, 64, 8, 16, 9, 1, 1, 0, b.BF16, 1)     # K > 8
    assert b.lib.c2r_route(C.byref(bad), None, None, None, None, None, None, None, None) == -2


@pytest.mark.parametrize("E,P", [(8, 2), (16, 4), (60, 4), (60, 8), (7, 3), (5, 5), (9, 1)])
def test_place_experts_matches_oracle(b, E, P):
    idx, _ = O.topk_route(G.random_logits(E * 31 + P, 2000, E), min(4, E))
    Cm = O.collab_count(idx, E)
    cfg = b.make_config(1, 8, E, 16, 1, 0, P, 0, b.F32, 1)
    for mode, name in ((0, "greedy"), (1, "contiguous")):
        part = torch.zeros(E, dtype=torch.int32); rank = torch.zeros(E, dtype=torch.int32)
        b.place_experts(cfg, torch.from_numpy(Cm.astype(np.int32)), mode, part, rank)
        rp, rr = O.place_experts(Cm, P, mode=name)
        assert np.array_equal(part.numpy(), rp) and np.array_equal(rank.numpy(), rr)


def test_binding_refuses_to_import_without_library(tmp_path):
    import subprocess, sys
    code = ("import importlib.util, sys, os\n"
            f"src = open(os.path.join({ROOT!r}, 'paper_2504_01337_b200', 'binding.py')).read()\n"
            f"p = os.path.join({str(tmp_path)!r}, 'binding.py'); open(p, 'w').write(src)\n"
            "spec = importlib.util.spec_from_file_location('b', p)\n"
            "m = importlib.util.module_from_spec(spec)\n"
            "try:\n    spec.loader.exec_module(m)\nexcept ImportError as e:\n    print('REFUSED'); sys.exit(0)\nsys.exit(1)\n")
    out = subprocess.run([sys.executable, "-c", code], capture_output=True, text=True)
    assert out.returncode == 0 and "REFUSED" in out.stdout


def test_bench_accounting_matches_the_workload_arithmetic():
    """The numerators bench.py divides by measured time: algorithmic expert-GEMM flops per token
    (forward + backward = 3 x forward, padding not counted) for the three benchmark workloads."""
    import bench
    c3, c2, c5 = G.WORKLOADS["c3"], G.WORKLOADS["c2"], G.WORKLOADS["c5"]
    fwd_c3 = 6 * 4 * 2048 * 1408 + 6 * 2048 * 5632          # routed (K = 4) + shared expert
    assert bench.flops_per_token(c3) == 3 * fwd_c3 == 415_236_096
    assert bench.flops_per_token(c5) == bench.flops_per_token(c3)
    assert bench.flops_per_token(c2) == 3 * 6 * 4 * 4096 * 688
    # whole step at c3: 6.80 TFLOP, the figure the roofline line reports per 12 launches
    assert abs(bench.flops_per_token(c3) * c3.N / 1e12 - 6.803) < 1e-3
    # bandwidth-bound calls at c3, bytes per token: dispatch reads a 4 KiB row and writes it K = 4 times
    # (+ 64 B of index); the combine reads K + 1 rows (shared expert) and writes one -- in fp32 as stored
    # (4 * 5 * 2048 + 4096 B) or in the storage type (2 * 6 * 2048 B)
    moved, alg = bench.hbm_bytes(c3)
    assert moved["permute"] == c3.N * (5 * 4096 + 64) and alg["permute"] == moved["permute"]
    assert moved["combine"] == c3.N * (4 * 5 * 2048 + 4096) and alg["combine"] == c3.N * 2 * 6 * 2048
    assert moved["spread_dY"] == c3.N * 5 * 4096
    assert moved["gate_logits"] == c3.N * (4096 + 61 * 4) + 61 * 4096
