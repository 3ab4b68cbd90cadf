"""The d-sharded path with the CUDA kernels: two processes share one GPU, each holding its own column range of
the received matrix, the plan's projection and locator kernels on either side of the one exchange (all-reduce of
the 3 n-double projection record, here over gloo).  No kernel of one rank waits for the other: the exchange
happens on the host between two launches.  Flags and sums against the oracle on the whole matrix."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import draco_inputs as di
from oracle import draco_oracle as orc

pytestmark = pytest.mark.gpu


def _worker(rank, world, port, n, s, d, adv, result):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import paper_1803_09877_b200 as dr
    from paper_1803_09877_b200.sharding import locate_sharded, merge_flags, shard_range
    torch.cuda.set_device(0)
    c0, c1 = shard_range(d, world, rank)
    G = di.gradient_rows(7, n, d, i0=c0, i1=c1)
    R = orc.cyc_encode(G, n, s)                                    # this rank's columns of the complex64 vectors
    di.apply_adversaries(R, adv, [di.ADV_REVGRAD] * len(adv), [100.0] * len(adv), seed=9, i0=c0)
    f = di.projection_vector(8, d, i0=c0, i1=c1)
    plan = dr.Plan(n, s, c1 - c0, dr.CYC)
    Rd = torch.from_numpy(np.ascontiguousarray(R).view(np.float32)).cuda()
    fd = torch.from_numpy(f).cuda()
    flags = torch.zeros(n, dtype=torch.uint8, device="cuda")
    e = torch.zeros(3 * n, dtype=torch.float64, device="cuda")
    locate_sharded(plan, Rd, fd, flags, e)
    u = torch.empty(c1 - c0, dtype=torch.float32, device="cuda")
    plan.decode(Rd, flags, u)
    info = plan.info()
    # repetition code on the same ranks: every rank decodes its columns, the flags are OR-ed
    rplan = dr.Plan(n, s, c1 - c0, dr.REP)
    Zr = orc.rep_encode(G, n, s)
    if rank == 1:
        Zr[adv[0], 5] += np.float32(1.0)                           # one corrupted entry, seen by rank 1 only
    rflags = torch.zeros(n, dtype=torch.uint8, device="cuda")
    ru = torch.empty(c1 - c0, dtype=torch.float32, device="cuda")
    rplan.locate_decode(torch.from_numpy(Zr).cuda(), None, rflags, ru)
    merge_flags(rflags)
    torch.cuda.synchronize()
    result[rank] = (flags.cpu().numpy(), e.cpu().numpy(), u.cpu().numpy(), (c0, c1), info["status"], rflags.cpu().numpy(),
                    ru.cpu().numpy())
    dist.destroy_process_group()


def test_two_ranks_on_one_gpu_locate_over_the_exchange_and_decode_their_shards():
    n, s, d, world = 15, 2, 10_000, 2
    adv = [3, 11]
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    manager = mp.get_context("spawn").Manager()
    result = manager.dict()
    mp.spawn(_worker, args=(world, port, n, s, d, adv, result), nprocs=world, join=True)
    G = di.gradient_rows(7, n, d)
    R = orc.cyc_encode(G, n, s)
    di.apply_adversaries(R, adv, [di.ADV_REVGRAD] * 2, [100.0] * 2, seed=9)
    f = di.projection_vector(8, d)
    whole = orc.cyc_locate(R, f, n, s)
    assert sorted(np.flatnonzero(whole["flags"])) == adv
    uo = orc.cyc_decode(R, n, s, whole["flags"])
    qo = orc.cyc_project_energy(R)
    exact_rep = G.astype(np.float64).sum(axis=0)
    for r in range(world):
        flags, e, u, (c0, c1), status, rflags, ru = result[r]
        np.testing.assert_array_equal(flags.astype(bool), whole["flags"])
        assert status == 0
        # the summed record is the whole vector's: e to the order of fp64 additions, q likewise
        assert np.abs(e[: 2 * n].view(np.complex128) - whole["e"]).max() <= 1e-11 * np.sqrt(qo.max() * 2 * d)
        assert np.abs(e[2 * n:] - qo).max() <= 1e-12 * qo.max()
        assert np.abs(u - uo[c0:c1]).max() <= 1e-6 * np.abs(uo).max()
        assert sorted(np.flatnonzero(rflags)) == [adv[0]]           # seen by one shard, known to both
        assert np.abs(ru - exact_rep[c0:c1]).max() <= 1e-5 * np.abs(exact_rep).max()
    np.testing.assert_array_equal(result[0][1], result[1][1])      # every rank holds the same record
