"""The multi-process plumbing bench.py uses for N > 1, exercised with two gloo ranks on CPU."""
import os
import socket
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys
    sys.path.insert(0, %r)
    from paper_2310_01655_b200 import dist_util as du
    from paper_2310_01655_b200 import inputs as wl
    rank, world, local = du.env_rank()
    assert du.init("gloo")
    du.barrier()
    # the slowest rank sets the job's time
    ms = du.max_over_ranks(10.0 + 5.0 * rank)
    assert ms == 10.0 + 5.0 * (world - 1), ms
    # every rank draws its own batch
    w = wl.small_workload(B=1, H=1, n=128, r=16, b=128, dtype="f32", seed=3)
    wr = wl.Workload(**dict(w.asdict(), data_seed=du.rank_seed(w.data_seed, rank)))
    q = wl.make_inputs(wr, "cpu")["Q"]
    import torch, torch.distributed as dist
    sums = [torch.zeros(1, dtype=torch.float64) for _ in range(world)]
    dist.all_gather(sums, q.double().sum().reshape(1))
    assert len({round(float(s), 6) for s in sums}) == world, sums
    tput = du.aggregate_throughput(units_per_rank_step=1000, steps=4, max_ms=ms, world=world)
    assert abs(tput - world * 1000 * 4 / (ms / 1e3)) < 1e-6
    du.shutdown()
    print("rank", rank, "ok")
""") % ROOT


SEQ_WORKER = textwrap.dedent("""
    # A sequence cut over the ranks: every rank holds n / world consecutive rows of one head.  Its
    # rows' outputs are the causal result inside the shard plus phi'(Q_shard) times the sum of the
    # earlier shards' end states -- which is what exclusive_prefix_over_ranks delivers.
    import os, sys
    sys.path.insert(0, %r)
    import numpy as np, torch
    from paper_2310_01655_b200 import dist_util as du
    from oracle import polysketch as orc
    rank, world, local = du.env_rank()
    assert du.init("gloo")
    g = np.random.default_rng(7)                      # the same full problem on every rank
    n, h, r = 48, 6, 4
    Q, K, V = (g.standard_normal((n, h)) for _ in range(3))
    G1, G2 = g.standard_normal((h, r)), g.standard_normal((h, r))
    O_full, d_full = orc.causal_polysketch_attention(Q, K, V, G1, G2)
    lo, hi = rank * n // world, (rank + 1) * n // world
    Qs, Ks, Vs = Q[lo:hi], K[lo:hi], V[lo:hi]
    Vt = np.concatenate([Vs, np.ones((hi - lo, 1))], axis=1)
    total = orc.polysketch_non_negative(Ks, G1, G2).T @ Vt          # this shard's end state
    start = du.exclusive_prefix_over_ranks(torch.from_numpy(total)).numpy()
    if rank == 0:
        assert np.all(start == 0)
    W = orc.causal_weights(Qs, Ks, G1, G2)                           # pairs inside the shard
    N = W @ Vt + orc.polysketch_non_negative(Qs, G1, G2) @ start     # + everything before the shard
    d = 1.0 + N[:, h]
    np.testing.assert_allclose(d, d_full[lo:hi], rtol=1e-11)
    np.testing.assert_allclose(N[:, :h] / d[:, None], O_full[lo:hi], rtol=1e-10, atol=1e-12)
    du.shutdown()
    print("rank", rank, "ok")
""") % ROOT


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def test_two_gloo_ranks(tmp_path):
    _run_ranks(tmp_path, WORKER, 2)


def test_sequence_shards_exchange_their_end_states(tmp_path):
    _run_ranks(tmp_path, SEQ_WORKER, 2)
    _run_ranks(tmp_path, SEQ_WORKER, 3)


def _run_ranks(tmp_path, source, world):
    script = tmp_path / "worker.py"
    script.write_text(source)
    port = _free_port()
    procs = []
    for rank in range(world):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.STDOUT, text=True))
    outs = [p.communicate(timeout=240)[0] for p in procs]
    for rank, (p, out) in enumerate(zip(procs, outs)):
        assert p.returncode == 0, out
        assert "rank %d ok" % rank in out


def test_single_process_helpers():
    from paper_2310_01655_b200 import dist_util as du
    assert du.env_rank()[1] >= 1
    assert du.max_over_ranks(3.5) == 3.5
    assert du.rank_seed(5, 0) == 5 and du.rank_seed(5, 2) != du.rank_seed(5, 1)
    assert du.aggregate_throughput(10, 2, 1000.0, 4) == 80.0
