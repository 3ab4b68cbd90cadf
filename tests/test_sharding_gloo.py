"""The d-sharded path on two and three CPU ranks (gloo): the sharding helpers and the one exchange,
with the oracle standing in for the kernels behind the plan interface."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import draco_inputs as di
from oracle import draco_oracle as orc


def test_shard_range_covers_and_aligns():
    from paper_1803_09877_b200.sharding import shard_range
    for d, world in [(60_200_000, 8), (1001, 2), (2048, 4), (5000, 3), (1, 2)]:
        pieces = [shard_range(d, world, r) for r in range(world)]
        assert pieces[0][0] == 0 and pieces[-1][1] == d
        for (a0, a1), (b0, b1) in zip(pieces, pieces[1:]):
            assert a1 == b0 and a0 <= a1
        assert all(c0 % 2048 == 0 or c0 == d for c0, _ in pieces)
    with pytest.raises(ValueError):
        shard_range(10, 2, 2)


class _OraclePlan:
    """Same method names as paper_1803_09877_b200.Plan, computing with the oracle on CPU tensors."""

    def __init__(self, n, s):
        self.n, self.s = n, s

    def cyc_project(self, R, f, e, stream=None):
        Rc = R.numpy().view(np.complex64)
        val = orc.cyc_project(Rc, f.numpy())
        e[: 2 * self.n].copy_(torch.from_numpy(val.view(np.float64)))
        e[2 * self.n:].copy_(torch.from_numpy(orc.cyc_project_energy(Rc)))

    def cyc_locate_from_projection(self, e, flags, stream=None):
        out = orc.cyc_locate_from_projection(e.numpy()[: 2 * self.n].view(np.complex128), e.numpy()[2 * self.n:], self.n, self.s)
        flags.copy_(torch.from_numpy(out["flags"].astype(np.uint8)))


def _worker(rank, world, port, n, s, d, adv, result):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_1803_09877_b200.sharding import locate_sharded, merge_flags, shard_range
    c0, c1 = shard_range(d, world, rank)
    G = di.gradient_rows(7, n, d, i0=c0, i1=c1)
    R = orc.cyc_encode(G, n, s)
    di.apply_adversaries(R, adv, [di.ADV_REVGRAD] * len(adv), [100.0] * len(adv), seed=9, i0=c0)
    f = di.projection_vector(8, d, i0=c0, i1=c1)
    flags = torch.zeros(n, dtype=torch.uint8)
    e = torch.zeros(3 * n, dtype=torch.float64)
    locate_sharded(_OraclePlan(n, s), torch.from_numpy(R.view(np.float32)), torch.from_numpy(f), flags, e)
    u = orc.cyc_decode(R, n, s, flags.numpy().astype(bool))
    rep_flags = torch.zeros(n, dtype=torch.uint8)
    rep_flags[rank] = 1
    merge_flags(rep_flags)
    result[rank] = (flags.numpy().copy(), e.numpy().copy(), u, (c0, c1), rep_flags.numpy().copy())
    dist.destroy_process_group()


@pytest.mark.parametrize("world,d", [(2, 10_000), (3, 9_001)])       # 3 ranks: shards of 4096, 4096 and 809 coordinates
def test_sharded_locate_and_decode(world, d):
    n, s = 15, 2
    adv = [3, 11]
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    manager = mp.get_context("spawn").Manager()
    result = manager.dict()
    mp.spawn(_worker, args=(world, port, n, s, d, adv, result), nprocs=world, join=True)
    # single-process answer
    G = di.gradient_rows(7, n, d)
    R = orc.cyc_encode(G, n, s)
    di.apply_adversaries(R, adv, [di.ADV_REVGRAD] * 2, [100.0] * 2, seed=9)
    f = di.projection_vector(8, d)
    whole = orc.cyc_locate(R, f, n, s)
    for r in range(world):
        flags, e, u, (c0, c1), rep_flags = result[r]
        assert sorted(np.flatnonzero(flags)) == adv
        np.testing.assert_allclose(e[: 2 * n].view(np.complex128), whole["e"], rtol=1e-10, atol=1e-6 * whole["scale"])
        np.testing.assert_allclose(e[2 * n:], orc.cyc_project_energy(R), rtol=1e-10)
        exact = G[:, c0:c1].astype(np.float64).sum(axis=0)
        assert np.abs(u - exact).max() <= 1e-4 * np.abs(exact).max()
        assert rep_flags.tolist()[:world] == [1] * world and rep_flags.sum() == world
    for r in range(1, world):
        np.testing.assert_array_equal(result[0][1], result[r][1])      # every rank holds the same e
    sizes = [result[r][3][1] - result[r][3][0] for r in range(world)]
    assert sum(sizes) == d and (world == 2 or len(set(sizes)) > 1)     # the 3-rank case has uneven shards


def test_a_given_stream_is_made_current_around_the_collective(monkeypatch):
    """locate_sharded(stream=...) runs projection, all-reduce and solve with that stream as torch's current one
    (the collective is enqueued on the current stream, whatever stream the kernels were given)."""
    import contextlib

    from paper_1803_09877_b200 import sharding
    events = []

    @contextlib.contextmanager
    def fake_stream_ctx(stream):
        events.append(("enter", stream))
        yield
        events.append(("exit", stream))

    class RecordingPlan:
        def cyc_project(self, R, f, e, stream=None):
            events.append(("project", stream))

        def cyc_locate_from_projection(self, e, flags, stream=None):
            events.append(("solve", stream))

    monkeypatch.setattr(torch.cuda, "stream", fake_stream_ctx)
    token = object()
    flags = torch.zeros(4, dtype=torch.uint8)
    sharding.locate_sharded(RecordingPlan(), None, None, flags, None, stream=token)
    assert events == [("enter", token), ("project", token), ("solve", token), ("exit", token)]
    events.clear()
    sharding.merge_flags(flags, stream=token)
    assert events == [("enter", token), ("exit", token)]
    events.clear()
    sharding.locate_sharded(RecordingPlan(), None, None, flags, None)          # no stream: nothing is switched
    assert events == [("project", None), ("solve", None)]
