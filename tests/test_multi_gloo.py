"""The multi-GPU benchmark's host logic on CPU: two gloo ranks, each with its own seeded batch and
its own measured time; the whole-job figure uses the slowest rank's time."""
import os
import socket
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    from paper_2602_12128_b200 import multi
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    g = torch.Generator().manual_seed(multi.rank_seed(1000, rank))
    x = torch.randn(8, generator=g)
    ms = 2.0 + 3.0 * rank                       # rank 1 is the slow one
    slow = multi.max_over_ranks(ms, dist)
    gathered = [torch.zeros(8) for _ in range(world)]
    dist.all_gather(gathered, x)
    out.put((rank, slow, multi.whole_job_rate(100.0, world, slow), bool(torch.equal(gathered[0], gathered[1]))))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_max_time_and_distinct_batches():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, slow, rate, same in res:
        assert slow == pytest.approx(5.0)
        assert rate == pytest.approx(2 * 100.0 / 5e-3)
        assert not same


def test_single_process_needs_no_group():
    sys.path.insert(0, ROOT)
    from paper_2602_12128_b200 import multi
    assert multi.max_over_ranks(3.5) == 3.5
    assert multi.whole_job_rate(10.0, 1, 1000.0) == 10.0


def _shard_worker(rank, world, port, out):
    """Sequence sharding on the oracle: each rank builds the state of its own tokens, the ranks add them with the
    library's host helper, and every rank reads out its own tokens against the sum."""
    sys.path.insert(0, ROOT)
    import numpy as np
    from oracle import hla_oracle as orc
    from paper_2602_12128_b200 import multi
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    rng = np.random.default_rng(5)                      # the same full problem on every rank
    n, dphi, d, F = 37, 3, 4, 3
    q = np.abs(rng.standard_normal((n, dphi)))
    ks = [np.abs(rng.standard_normal((n, dphi))) for _ in range(F)]
    v = rng.standard_normal((n, d))
    do = rng.standard_normal((n, d))
    lo, hi = multi.shard_bounds(n, world, rank)
    C, z = orc.context_state([k[lo:hi] for k in ks], v[lo:hi])
    state = torch.from_numpy(np.concatenate([C, z[:, None]], axis=1))
    multi.all_reduce_sum(state, dist)
    Cs, zs = state.numpy()[:, :d], state.numpy()[:, d]
    o, eta = orc.readout(q[lo:hi], F, Cs, zs, 1e-3)
    o_full, eta_full = orc.hla_quadratic(q, ks, v, 1e-3)
    ok_fwd = bool(np.allclose(o, o_full[lo:hi], rtol=1e-10, atol=1e-12) and np.allclose(eta, eta_full[lo:hi], rtol=1e-10))
    # backward: the gradient state is a sum over the query tokens
    Tq = orc.outer_features([q[lo:hi]] * F)
    r = 1.0 / (eta + 1e-3)
    dnum = do[lo:hi] * r[:, None]
    deta = -r * np.sum(do[lo:hi] * o, axis=1)
    dstate = torch.from_numpy(np.concatenate([Tq.T @ dnum, (Tq.T @ deta)[:, None]], axis=1))
    multi.all_reduce_sum(dstate, dist)
    dC, dz = dstate.numpy()[:, :d], dstate.numpy()[:, d]
    Tk = orc.outer_features([k[lo:hi] for k in ks])
    dv = Tk @ dC
    _, _, dv_full = orc.hla_quadratic_backward(q, ks, v, do, 1e-3)
    ok_bwd = bool(np.allclose(dv, dv_full[lo:hi], rtol=1e-9, atol=1e-12)) and dz.shape == (dphi ** F,)
    out.put((rank, lo, hi, ok_fwd, ok_bwd))
    dist.barrier()
    dist.destroy_process_group()


def test_sequence_sharding_state_sum_two_ranks():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_shard_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [(r[1], r[2]) for r in res] == [(0, 19), (19, 37)]       # 37 tokens over two ranks: 19 + 18
    assert all(r[3] and r[4] for r in res)


def _causal_shard_worker(rank, world, port, out):
    """Causal sequence sharding on the oracle: each rank builds the state of its own tokens, the library's host helper
    gives it the state of the tokens before its shard (an exclusive prefix over the ranks), and the rank's causal
    outputs follow from its own sequential pass plus that state (the pass is linear in the state it starts from)."""
    sys.path.insert(0, ROOT)
    import numpy as np
    from oracle import hla_oracle as orc
    from paper_2602_12128_b200 import multi
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    rng = np.random.default_rng(11)                     # the same full problem on every rank
    n, dphi, d, F, eps = 41, 3, 4, 3, 1e-3
    q = np.abs(rng.standard_normal((n, dphi)))
    ks = [np.abs(rng.standard_normal((n, dphi))) for _ in range(F)]
    v = rng.standard_normal((n, d))
    lo, hi = multi.shard_bounds(n, world, rank)
    C, z = orc.context_state([k[lo:hi] for k in ks], v[lo:hi])
    local = torch.from_numpy(np.concatenate([C, z[:, None]], axis=1))
    before = multi.exclusive_prefix_state(local, dist).numpy()
    if lo > 0:
        Cb, zb = orc.context_state([k[:lo] for k in ks], v[:lo])
    else:
        Cb, zb = np.zeros_like(C), np.zeros_like(z)
    ok_prefix = bool(np.allclose(before[:, :d], Cb, rtol=1e-12, atol=1e-12) and np.allclose(before[:, d], zb, rtol=1e-12, atol=1e-12))
    o_loc, eta_loc = orc.hla_streaming(q[lo:hi], [k[lo:hi] for k in ks], v[lo:hi], eps)
    Tq = orc.outer_features([q[lo:hi]] * F)
    eta = eta_loc + Tq @ before[:, d]
    o = (o_loc * (eta_loc + eps)[:, None] + Tq @ before[:, :d]) / (eta + eps)[:, None]
    o_full, eta_full = orc.hla_quadratic_causal(q, ks, v, eps)
    ok_out = bool(np.allclose(o, o_full[lo:hi], rtol=1e-9, atol=1e-12) and np.allclose(eta, eta_full[lo:hi], rtol=1e-10))
    out.put((rank, lo, hi, ok_prefix, ok_out))
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.parametrize("world", [2, 3])
def test_causal_sequence_sharding_exclusive_prefix(world):
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_causal_shard_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert res[0][1] == 0 and res[-1][2] == 41 and all(res[i][2] == res[i + 1][1] for i in range(world - 1))
    assert all(r[3] and r[4] for r in res)


def test_shard_bounds_cover_the_sequence():
    sys.path.insert(0, ROOT)
    from paper_2602_12128_b200 import multi
    for n in (1, 7, 128, 32760):
        for world in (1, 2, 3, 8):
            b = [multi.shard_bounds(n, world, r) for r in range(world)]
            assert b[0][0] == 0 and b[-1][1] == n
            assert all(b[i][1] == b[i + 1][0] for i in range(world - 1))
            sizes = [hi - lo for lo, hi in b]
            assert max(sizes) - min(sizes) <= 1
