"""No-GPU checks: the built library loads, exports every symbol the header declares, and its
host-only entry points agree with the oracle's rules; sequence sharding over gloo ranks."""
import os
import re
import subprocess
import sys

import pytest

import oracle

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    from paper_2605_17447_b200 import _lib, build
    build.build()
    header = open(os.path.join(ROOT, "include", "fastocr.h")).read()
    declared = set(re.findall(r"\b(fastocr_[a-z_]+)\s*\(", header))
    assert {"fastocr_focal_scores", "fastocr_select_topk", "fastocr_sparse_decode_attn",
            "fastocr_dense_decode_attn", "fastocr_decode_step"} <= declared
    lib = _lib.load()
    for name in declared:
        assert hasattr(lib, name), name
    assert declared == set(_lib.EXPORTS), declared ^ set(_lib.EXPORTS)


def test_host_rules_agree_with_oracle():
    import paper_2605_17447_b200 as fo
    for n in (0, 1, 20, 77, 1000, 1024, 4096, 8192, 16384, 32768):
        for tau in (0.0, 0.004, 0.02, 0.05, 0.1, 0.2, 0.25, 1.0, 1.5):
            assert fo.kept_count(n, tau) == oracle.kept_count(n, tau), (n, tau)
    import random
    rnd = random.Random(4)
    for _ in range(200):
        L = rnd.randint(1, 40)
        r = [rnd.choice([0.1, 0.2, 0.3, rnd.random()]) for _ in range(L)]
        rho, gap = rnd.choice([0.05, 0.1, 0.2, 0.5, 1.0]), rnd.randint(0, 4)
        assert fo.focal_layers(r, rho, gap) == oracle.focal_layers(r, rho, gap)
    assert abs(fo.attn_flops(8, 36, 2048, 4096) - oracle.attn_flops(8, 36, 2048, 4096)) < 1.0
    for b, l, h, s_, f, sk in ((8, 36, 2048, 4096, 4, 204.8), (4, 36, 2048, 8192, 3, 409.6), (64, 28, 3584, 8449, 2, 666), (1, 5, 64, 100, 0, 0)):
        want = oracle.attn_flops_pruned(b, l, h, s_, f, sk)
        assert abs(fo.attn_flops_pruned(b, l, h, s_, f, sk) - want) <= 1e-9 * want


def test_product_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2605_17447_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".h", ".cuh")):
                assert "oracle" not in open(os.path.join(dirpath, f)).read().lower().replace("no cpu or pytorch", ""), f


_GLOO_WORKER = r"""
import os, sys, torch, torch.distributed as dist
sys.path.insert(0, os.environ["FASTOCR_ROOT"])
from paper_2605_17447_b200.sharding import shard_sequences
dist.init_process_group("gloo", init_method="tcp://127.0.0.1:%s" % os.environ["PORT"],
                        rank=int(os.environ["RANK"]), world_size=int(os.environ["WORLD_SIZE"]))
B = 33
lo, hi = shard_sequences(B, dist.get_rank(), dist.get_world_size())
own = torch.zeros(B, dtype=torch.int64); own[lo:hi] = 1
units = torch.tensor([float(hi - lo)]); t = torch.tensor([1.0 + dist.get_rank()])
dist.all_reduce(own); dist.all_reduce(units); dist.all_reduce(t, op=dist.ReduceOp.MAX)
assert own.tolist() == [1] * B, own          # every sequence owned exactly once
assert units.item() == B and t.item() == dist.get_world_size()
dist.barrier(); dist.destroy_process_group()
"""


def test_sequence_sharding_world_size_two_gloo(tmp_path):
    import socket
    s = socket.socket(); s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]; s.close()
    script = tmp_path / "w.py"
    script.write_text(_GLOO_WORKER)
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), WORLD_SIZE="2", PORT=str(port), FASTOCR_ROOT=ROOT)
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env))
    for p in procs:
        assert p.wait(timeout=120) == 0


def test_shard_sequences_edges():
    from paper_2605_17447_b200.sharding import shard_sequences
    assert [shard_sequences(5, r, 8) for r in range(8)] == [(0, 1), (1, 2), (2, 3), (3, 4), (4, 5), (5, 5), (5, 5), (5, 5)]
    assert shard_sequences(64, 3, 8) == (24, 32)
    with pytest.raises(ValueError):
        shard_sequences(4, 2, 2)
