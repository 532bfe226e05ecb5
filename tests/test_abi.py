"""The C-ABI library loads and exports every entry point that include/cdb.h declares (no compute)."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "cdb.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(cdb_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_entry_point():
    import __graft_entry__
    __graft_entry__.build()
    from paper_2608_09444_b200 import binding
    names = declared_symbols()
    assert len(names) >= 16
    lib = ctypes.CDLL(os.path.join(ROOT, "paper_2608_09444_b200", "libcdb.so"))
    for n in names:
        assert hasattr(lib, n), n
    assert set(binding.EXPORTS) == set(names)                     # the binding wraps exactly what the header declares


def test_struct_sizes_match_the_header():
    from paper_2608_09444_b200 import binding
    assert ctypes.sizeof(binding.Config) == 18 * 4 + 4 * 4 + 4
    assert ctypes.sizeof(binding.Weights) == 11 * 8
    assert ctypes.sizeof(binding.RowsStruct) == 4 + 4 + 6 * 8 + 4 + 4 + 8 # int, pad, six pointers, int, pad, pointer


def test_null_handle_is_an_error_not_a_crash():
    from paper_2608_09444_b200 import binding
    assert binding.lib.cdb_destroy(None) == 0
    assert binding.lib.cdb_set_gate(None, 0.0, 0.0) == binding.ERR_ARG
    assert binding.lib.cdb_poll_status(None, None) == binding.ERR_ARG
    assert binding.lib.cdb_last_error(None) == b"invalid handle"


def test_kv_footprint_accounting_matches_table1():
    """The driver's KV accounting against the sizes printed in the paper's Table 1 (appendix C.1): what the page
    pools reserve per cached token equals the table in every row once the prelude and coda layers have a page space
    of their own; with one page space for all layers it exceeds the table for boundary layers with several slots."""
    import os
    from paper_2608_09444_b200 import synth
    from paper_2608_09444_b200.engine import kv_footprint
    dims = {"ouro": synth.OURO_1P4B, "huginn": synth.HUGINN_3P5B}
    golden = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "table1_kv_footprint.txt")
    for line in open(golden):
        if line.startswith("#") or not line.strip():
            continue
        model, slots, kib, gib = line.split()
        used, reserved = kv_footprint(dims[model], int(slots))
        assert abs(used / 1024 - float(kib)) <= 0.5 and abs(used * 4096 / 2**30 - float(gib)) <= 0.006
        assert reserved == used
        used1, reserved1 = kv_footprint(dims[model], int(slots), split_kv=False)
        assert used1 == used and reserved1 >= used and (reserved1 == used) == (model == "ouro" or int(slots) == 1)


def test_engines_reject_unknown_scheduling_modes_before_touching_the_gpu():
    import pytest
    from paper_2608_09444_b200 import synth
    from paper_2608_09444_b200.engine import Engine
    with pytest.raises(ValueError, match="unknown scheduling mode"):
        Engine(synth.TINY, None, max_batch=4, max_live=4, max_len=32, n_pages=8, mode="none")


def test_flop_bound_and_the_early_rejoin_rule_on_the_two_model_shapes():
    """Eq. 2 on the paper's shapes: F0 / Fr = 0.082 for the Ouro shape (LM head against one pass of the 24-layer core),
    the bound is 1 at full depth and (F0 + R Fr) / (F0 + dbar Fr) below it.  The pipelined engine's rule for letting
    tokens rejoin before the next step compares the rows that rejoin with the boundary cost in steps: cheap for the
    Ouro shape, never worth it for the Huginn shape."""
    from paper_2608_09444_b200 import synth
    from paper_2608_09444_b200.engine_async import boundary_cost_in_steps
    from paper_2608_09444_b200.offline import flop_bound
    ouro, hug = synth.OURO_1P4B, synth.HUGINN_3P5B
    f0 = ouro.V * ouro.d / (ouro.L_core * (4 * ouro.d ** 2 + 3 * ouro.d * ouro.F))
    assert abs(f0 - 0.082) < 5e-4
    assert flop_bound(ouro, ouro.R) == 1.0
    assert abs(flop_bound(ouro, 2.5) - (f0 + 4) / (f0 + 2.5)) < 1e-12
    assert abs(flop_bound(hug, 12.0) - 2.51) < 0.01
    assert boundary_cost_in_steps(ouro) == 2 * f0 and boundary_cost_in_steps(ouro) < 0.2
    assert boundary_cost_in_steps(hug) > 1.0


def test_reference_arm_of_the_bench_runs_on_the_host_alone_and_prints_the_contract_line():
    """`bench.py --impl reference` times the CPU oracle on a bounded sample and needs neither a GPU nor the library: its
    process must not load libcdb.so, and its single JSON line carries the keys the benchmark contract names."""
    import json
    import os
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    code = ("import runpy, sys; sys.argv = ['bench.py', '--impl', 'reference', '--steps', '1', '--warmup', '0', '--layers', '1'];\n"
            "try:\n    runpy.run_path('bench.py', run_name='__main__')\nexcept SystemExit:\n    pass\n"
            "print('LIBCDB_LOADED' if 'libcdb' in open('/proc/self/maps').read() else 'LIBCDB_ABSENT')")
    out = subprocess.run([sys.executable, "-c", code], cwd=root, capture_output=True, text=True, timeout=600)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.strip()]
    assert lines[-1] == "LIBCDB_ABSENT"
    line = json.loads(lines[-2])
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                "vs_baseline", "dtype", "data", "config", "cpu_baseline", "e2e"):
        assert key in line, key
    assert line["impl"] == "reference" and line["metric"] == "token_loop_steps_per_s" and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["value"] == line["value"]
    assert line["e2e"]["value"] == line["value"] and line["e2e"]["h2d_bytes_per_step"] == 0
    assert "workload" in line["config"] and "model" not in line["config"]
