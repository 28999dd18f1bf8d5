"""CPU-side checks of the boundary: the C-ABI library loads and exports every entry point that
include/mw.h declares, the binding mirrors them, and the benchmark's multi-rank bookkeeping works."""
import ctypes
import os
import re
import socket
import sys

import pytest

from paper_2605_22428_b200 import binding as mw
from paper_2605_22428_b200 import build as mwbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_entry_points():
    text = open(os.path.join(ROOT, "include", "mw.h")).read()
    return re.findall(r"^MW_API\s+[\w\s\*]+?\b(mw_\w+)\s*\(", text, flags=re.M)


def test_library_builds_and_exports_every_declared_symbol():
    path = mwbuild.build_library()
    assert os.path.exists(path)
    lib = ctypes.CDLL(path)
    names = declared_entry_points()
    assert len(names) >= 11 and "mw_plan" in names and "mw_dispatch" in names and "mw_allgather_pack" in names
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(names) == sorted(mw.EXPORTS)


def test_header_is_plain_c_and_struct_layouts_match_the_binding(tmp_path):
    """include/mw.h must compile as C99 on its own (no C++, no CUDA or torch types), and the structs the binding
    mirrors with ctypes must have the sizes the C compiler gives them."""
    import subprocess
    header = os.path.join(ROOT, "include", "mw.h")
    subprocess.check_call(["gcc", "-std=c99", "-Wall", "-Werror", "-fsyntax-only", "-x", "c", header])
    src = tmp_path / "sizes.c"
    src.write_text('#include <stdio.h>\n#include "mw.h"\nint main(void) { printf("%zu %zu %zu\\n", sizeof(mw_config), '
                   'sizeof(mw_totals), sizeof(mw_plan_view)); return 0; }\n')
    exe = tmp_path / "sizes"
    subprocess.check_call(["gcc", "-std=c99", "-I", os.path.join(ROOT, "include"), str(src), "-o", str(exe)])
    got = [int(v) for v in subprocess.check_output([str(exe)]).split()]
    assert got == [ctypes.sizeof(mw.mw_config), ctypes.sizeof(mw.mw_totals), ctypes.sizeof(mw.mw_plan_view)]


def test_error_strings_and_struct_sizes():
    assert mw.strerror(mw.MW_OK) == "ok"
    for code in range(-7, 0):
        assert mw.strerror(code) != "unknown error code"
    assert ctypes.sizeof(mw.mw_totals) == 64 and ctypes.sizeof(mw.mw_config) == 40
    assert ctypes.sizeof(mw.mw_plan_view) == 12 * 8 + 16


def test_binding_fails_loudly_without_the_library(monkeypatch, tmp_path):
    monkeypatch.setattr(mw, "_lib", None)
    monkeypatch.setattr(mwbuild, "LIB_PATH", str(tmp_path / "libmw.so"))
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        mw.lib()


def test_product_code_does_not_touch_the_oracle():
    pkg = os.path.join(ROOT, "paper_2605_22428_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert not re.search(r"(from|import)\s+oracle|\bmwo\b|libmwo|oracle/", text), f


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out):
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    import torch
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    total, e2e, units = bench.aggregate_over_ranks(dist, 10.0 + rank, 100.0 - rank, 1000.0 * (rank + 1), torch.device("cpu"))
    out.put((rank, total, e2e, units))
    dist.destroy_process_group()


def test_replica_aggregation_two_ranks_gloo():
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, total, e2e, units in got:
        assert total == 11.0 and e2e == 100.0 and units == 3000.0     # max time, max time, summed work


def test_plain_start_with_gpus_2_launches_two_ranks():
    """`bench.py --gpus 2` started without a launcher starts the ranks itself; here on the CPU (gloo), figures made up."""
    import json
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--selftest-aggregate"],
                         capture_output=True, text=True, timeout=300, check=True, env=env).stdout.strip()
    line = json.loads(out.splitlines()[-1])
    assert line == {"selftest": "aggregate", "n_gpus": 2, "total_ms": 11.0, "e2e_ms": 100.0, "units": 3000.0}


def test_all_core_leg_of_the_cpu_baseline_moves_the_same_bytes():
    """The benchmark's all-core leg runs the oracle's own pack / deliver on slices of the send rows from several threads:
    the buffers must equal those of the plain single call."""
    import numpy as np
    sys.path.insert(0, ROOT)
    import bench
    from paper_2605_22428_b200 import workloads as wl
    inp = wl.make_dispatch("dsv3_prefill", T=777, H=40)
    one = bench.oracle_stages(inp, inp.shape.R, inp.shape.row_bytes, keep=True)
    many = bench.oracle_stages(inp, inp.shape.R, inp.shape.row_bytes, threads=5, keep=True)
    assert one[3] == many[3]
    assert np.array_equal(one[4], many[4]) and np.array_equal(one[5].reshape(-1), many[5].reshape(-1))


def test_reference_arm_prints_one_json_line():
    import json
    import subprocess
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                          "--warmup", "0"], capture_output=True, text=True, timeout=300, check=True).stdout.strip()
    line = json.loads(out.splitlines()[-1])
    assert line["impl"] == "reference" and line["unit"] == "GB/s" and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
