"""The N > 1 host logic on CPU: two gloo ranks agree on the controller's ratio,
reduce step times to the slowest rank, and lay out an all-gather buffer of
equal-size payloads that the oracle can sum."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2506_16235_b200 import build as nsml_build

nsml_build.build()


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import paper_2506_16235_b200 as nsml
    from paper_2506_16235_b200 import dp

    n, bits = 50_000, 16
    # every rank runs its own controller on its own (different) measurements; rank 0's ratio wins
    ctrl = nsml.Controller(startup_max_steps=0, ratio_init=0.2)
    ctrl.select_ratio(0, 0, 4.0 * n)
    mine = ctrl.select_ratio(1e5 if rank == 0 else 1e4, 1e-3 * (1 + rank), 4.0 * n)  # rank 1 sees a congested link
    ratio = dp.agree_ratio(mine)
    slowest = dp.max_over_ranks(10.0 + rank)
    # equal ratio -> equal payload size -> one fixed-size all-gather
    rng = np.random.default_rng(100 + rank)
    g = rng.standard_normal(n).astype(np.float32)
    p = oracle.compress(g, ratio, bits)
    raw = torch.from_numpy(nsml.pack_payload(n, bits, p.idx, half=p.half))
    assert raw.numel() == nsml.nsml_payload_bytes(n, ratio, bits)
    slots, total = dp.payload_slots(world, raw.numel())
    buf, gathered = dp.exchange_payloads(raw)  # the one fixed-size all-gather of the sparse path
    assert buf.numel() == total and torch.equal(gathered[rank], raw)
    assert all(v.data_ptr() % 16 == 0 for v in gathered)
    parts = [nsml.unpack_payload(t) for t in gathered]
    payloads = [oracle.Payload(n=n, k=q["k"], bits=bits, idx=q["idx"], raw=oracle.f16_bits_to_f32(q["half"]), half=q["half"])
                for q in parts]
    dense = oracle.decompress_sum(payloads, n)
    out[rank] = dict(mine=mine, ratio=ratio, slowest=slowest, checksum=float(np.abs(dense.astype(np.float64)).sum()),
                     slots=slots, total=total, k=[q["k"] for q in parts])
    dist.destroy_process_group()


def test_two_ranks_agree_and_sum():
    world, port = 2, _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0]["mine"] != res[1]["mine"]  # the ranks measured different transfer times
    assert res[0]["ratio"] == res[1]["ratio"] == res[0]["mine"]
    assert res[0]["slowest"] == res[1]["slowest"] == 11.0
    assert res[0]["checksum"] == res[1]["checksum"] > 0  # both ranks reconstruct the same dense sum
    assert res[0]["k"][0] == res[0]["k"][1]
    (a0, a1), (b0, b1) = res[0]["slots"]
    assert a0 == 0 and b0 % 16 == 0 and b0 >= a1 and res[0]["total"] >= b1


def _exchange_worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import paper_2506_16235_b200 as nsml
    from paper_2506_16235_b200 import dp

    # the loop the benchmark's exchange leg runs, with the CPU restatement standing in for the CUDA calls:
    # controller -> agreed ratio -> compress -> all-gather -> sum, the measured transfer fed back
    n, bits, steps = 30_000, 8, 5
    ctrl = nsml.Controller(startup_max_steps=0, ratio_init=0.04 if rank == 0 else 0.5)  # rank 1's own choice must not matter
    rng = np.random.default_rng(7 + rank)
    last, ratios, sent, sums = (0.0, 0.0), [], [], []
    for step in range(steps):
        g = rng.standard_normal(n).astype(np.float32)
        dense = {}

        def compress(ratio, g=g):
            p = oracle.compress(g, ratio, bits)
            return torch.from_numpy(nsml.pack_payload(n, bits, p.idx, codes=p.codes, scales=p.scales))

        def accumulate(views, dense=dense):
            parts = [nsml.unpack_payload(v) for v in views]
            ps = [oracle.Payload(n=n, k=q["k"], bits=bits, idx=q["idx"], raw=np.zeros(0, np.float32), codes=q["codes"],
                                 scales=q["scales"]) for q in parts]
            dense["sum"] = oracle.decompress_sum(ps, n)

        ratio, phases, last = dp.exchange_round(ctrl, last, 4.0 * n * world, compress, accumulate, on_cuda=False)
        assert len(phases) == 3 and all(ms >= 0.0 for ms in phases)
        assert last[0] == world * nsml.nsml_payload_bytes(n, ratio, bits) and last[1] == max(phases[1] * 1e-3, 1e-9)
        ratios.append(ratio)
        sent.append(last)
        sums.append(float(np.abs(dense["sum"].astype(np.float64)).sum()))
    out[rank] = dict(ratios=ratios, sent=sent, sums=sums, calls=ctrl.state().calls)
    dist.destroy_process_group()


def test_exchange_rounds_feed_the_controller_with_the_measured_transfer():
    world, port = 2, _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_exchange_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0]["ratios"] == res[1]["ratios"]          # every step both ranks compress at rank 0's ratio
    assert res[0]["ratios"][0] == 0.04                   # rank 0's initial ratio, not rank 1's 0.5
    assert len(set(res[0]["ratios"])) > 1                # and the controller moved it as transfers were measured
    assert res[0]["sent"] == res[1]["sent"]              # MAX-reduced times: both ranks feed the same measurement
    assert res[0]["sums"] == res[1]["sums"]              # both ranks reconstruct the same dense sums
    assert res[0]["calls"] == res[1]["calls"] == 5


def test_whole_job_value_is_the_aggregate():
    from paper_2506_16235_b200 import dp

    assert dp.whole_job_gbps(world=4, steps=10, bytes_per_rank_step=1e9, slowest_ms=1000.0) == 40.0
    assert dp.agree_ratio(0.25) == 0.25 and dp.max_over_ranks(3.5) == 3.5  # single process: identity
