"""World-size-2 run of the sharding logic on CPU (gloo): batch and head shards computed by separate ranks with no
exchange equal the unsharded result; a sequence cut along time, with the Conv1D history and each share's affine step
exchanged once, equals the uncut result; the step-time reduction is a maximum; rank seeds differ."""
import os
import socket
import subprocess
import sys

from paper_2402_19427_b200 import sharding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_split_range_covers_everything_once():
    for n in (1, 5, 8, 10, 512):
        for world in (1, 2, 3, 8):
            spans = [sharding.split_range(n, world, r) for r in range(world)]
            assert spans[0][0] == 0 and sum(c for _, c in spans) == n
            for (s0, c0), (s1, _) in zip(spans, spans[1:]):
                assert s0 + c0 == s1
            assert max(c for _, c in spans) - min(c for _, c in spans) <= 1


def test_two_gloo_ranks_shard_without_exchange(oracle):
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr", "127.0.0.1",
           "--master-port", str(port), os.path.join(ROOT, "tests", "multirank_worker.py")]
    env = dict(os.environ, OMP_NUM_THREADS="2")
    r = subprocess.run(cmd, capture_output=True, text=True, timeout=240, env=env, cwd=ROOT)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-2000:]
    assert "MULTIRANK_OK" in r.stdout


def test_affine_steps_compose_associatively():
    import numpy as np
    rng = np.random.default_rng(0)
    s = [(rng.uniform(0, 1, 7), rng.standard_normal(7)) for _ in range(3)]
    left = sharding.combine_steps(sharding.combine_steps(s[0], s[1]), s[2])
    right = sharding.combine_steps(s[0], sharding.combine_steps(s[1], s[2]))
    np.testing.assert_allclose(left[0], right[0], rtol=1e-14); np.testing.assert_allclose(left[1], right[1], rtol=1e-13)
    h = rng.standard_normal(7)
    step = h
    for a, b in s:
        step = a * step + b
    np.testing.assert_allclose(left[0] * h + left[1], step, rtol=1e-13)
    one = sharding.combine_steps((np.ones(7), np.zeros(7)), s[0])
    assert np.array_equal(one[0], s[0][0]) and np.array_equal(one[1], s[0][1])
