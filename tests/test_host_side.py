"""CPU-only checks of everything around the kernels: the library exports what the header
declares, the input generator is deterministic and in range, and the multi-rank
bookkeeping of the benchmark works over gloo with two ranks."""
import ctypes
import os
import re
import subprocess
import sys

import numpy as np
import pytest

import workloads as W

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    from paper_2605_16867_b200.build import build_library
    lib = ctypes.CDLL(build_library())
    header = open(os.path.join(ROOT, "include", "goodserve.h")).read()
    declared = re.findall(r"GS_API[^;(]*?\b(gs_[a-z_]+)\s*\(", header)
    assert len(declared) >= 12 and len(set(declared)) == len(declared)
    for name in declared:
        assert hasattr(lib, name), f"{name} is declared in goodserve.h but not exported"
    lib.gs_strerror.restype = ctypes.c_char_p
    assert b"aligned" in lib.gs_strerror(-4)
    assert lib.gs_strerror(12345) is not None


def test_binding_fails_loudly_without_a_gpu():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    from paper_2605_16867_b200 import GoodServe
    with pytest.raises(RuntimeError):
        GoodServe(0)


def test_product_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2605_16867_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text.lower(), f"{f} mentions the oracle"


def test_workload_shapes_ranges_and_determinism():
    for cfg_id, cfg in W.CONFIGS.items():
        n, a = min(cfg.n_requests, 5000), min(cfg.n_active, 5000)
        w1 = W.make_workload(cfg_id, n_requests=n, n_active=a)
        w2 = W.make_workload(cfg_id, n_requests=n, n_active=a)
        for c1, c2 in zip(w1.requests.columns() + w1.active.columns() + w1.instances.columns(),
                          w2.requests.columns() + w2.active.columns() + w2.instances.columns()):
            assert c1.tobytes() == c2.tobytes()
        r, act, inst = w1.requests, w1.active, w1.instances
        assert r.prompt_len.dtype == np.int32 and r.slo_ms.dtype == np.float32
        assert 16 <= r.prompt_len.min() and r.prompt_len.max() <= 16384
        assert 8 <= r.pred_decode_len.min() and r.pred_decode_len.max() <= 8192
        assert (r.slo_ms > 0).all()
        assert inst.n_instances == cfg.n_instances and w1.types.n_types == cfg.n_types
        assert (inst.type_id == np.arange(cfg.n_instances) % cfg.n_types).all()
        assert 0 <= inst.decode_batch.min() and inst.decode_batch.max() <= 64
        assert inst.free_kv_tokens.max() <= 200000 and inst.queued_prefill_tokens.max() <= 20000
        assert (act.generated_tokens <= act.pred_len).all() and (act.generated_tokens >= 0).all()
        assert (act.elapsed_ms <= act.slo_ms).all()
        assert 0 <= act.assigned_inst.min() and act.assigned_inst.max() < cfg.n_instances
        # growing N keeps the prefix (per-column streams)
        w3 = W.make_workload(cfg_id, n_requests=n + 100, n_active=a)
        assert (w3.requests.prompt_len[:n] == r.prompt_len).all()
    # config 0 uses the unperturbed constants
    t0 = W.make_workload(0).types
    np.testing.assert_allclose(t0.prefill_ms_per_tok, [1 / 40, 1 / 20, 1 / 10], rtol=1e-6)
    np.testing.assert_allclose(t0.tpot_a_ms, [8, 14, 25])
    # rounds of a stream differ
    w4 = W.make_workload(4, n_requests=1000, n_active=10)
    assert not (W.make_round_requests(w4, 1, 1000).prompt_len == w4.requests.prompt_len).all()
    assert (W.make_round_requests(w4, 0, 1000).prompt_len == w4.requests.prompt_len).all()


_GLOO_CHILD = r"""
import os, sys
sys.path.insert(0, {root!r})
import torch.distributed as dist
import bench
dist.init_process_group("gloo", init_method="tcp://127.0.0.1:{port}", rank=int(sys.argv[1]), world_size=2)
rank = dist.get_rank()
ms, units = bench.aggregate_over_ranks(10.0 + 5.0 * rank, 100.0 * (rank + 1), dist)
assert ms == 15.0 and units == 300.0, (ms, units)
assert bench.rank_seed(3, rank) == 3 + 1000 * rank
dist.barrier()
dist.destroy_process_group()
print("ok", rank)
"""


def test_two_rank_aggregation_over_gloo(tmp_path):
    import socket
    s = socket.socket(); s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]; s.close()
    script = tmp_path / "child.py"
    script.write_text(_GLOO_CHILD.format(root=ROOT, port=port))
    procs = [subprocess.Popen([sys.executable, str(script), str(r)], stdout=subprocess.PIPE,
                              stderr=subprocess.STDOUT, text=True) for r in range(2)]
    outs = [p.communicate(timeout=180)[0] for p in procs]
    for p, o in zip(procs, outs):
        assert p.returncode == 0, o
    # different seeds per rank give different batches of the same shape
    a = W.make_workload(1, seed=1, n_requests=100, n_active=10)
    b = W.make_workload(1, seed=1001, n_requests=100, n_active=10)
    assert a.requests.n == b.requests.n and not (a.requests.prompt_len == b.requests.prompt_len).all()


def test_reference_arm_prints_one_json_line():
    import json
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "1",
                          "--steps", "2", "--warmup", "1"], capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["value"] > 0 and line["cpu_baseline"]["kind"] == "oracle"
