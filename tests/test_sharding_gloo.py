"""The N > 1 host-side path on CPU: two gloo ranks split the independent (batch, KV head)
units, each rank works on its own shard with no data-path collective, and the only
exchanges are the barrier and the max-over-ranks reduction of the timing, as in bench.py.
The per-rank work here is the CPU oracle (no GPU in this test)."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2602_03152_b200 import synth


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _rank_main(rank, world, port, ret):
    from oracle import fasa_oracle as O

    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = synth.CONFIGS["c2"].replace(batch=3, n_q_heads=12, n_kv_heads=3, max_len=300, len_lo=100, len_hi=300, budget=32)
    t = synth.make_inputs(w, "cpu")
    units = synth.shard_units(w.batch * w.n_kv_heads, rank, world)
    G = w.group
    outs = torch.zeros((w.batch, w.n_q_heads, 128), dtype=torch.float64)
    for u in units:
        b, h = divmod(u, w.n_kv_heads)
        r = O.decode_bf16(synth.bf16_bits(t["q"][b:b + 1, h * G:(h + 1) * G]), synth.bf16_bits(t["k"][b:b + 1, h:h + 1]),
                          synth.bf16_bits(t["v"][b:b + 1, h:h + 1]), t["seq_lens"][b:b + 1].numpy(),
                          t["dom"][h:h + 1].numpy(), budget=w.budget, n_threads=1, want_dense=False)
        outs[b, h * G:(h + 1) * G] = torch.from_numpy(r["out"][0])
    dist.barrier()
    # timing reduction: max over ranks of a per-rank duration
    tt = torch.tensor([10.0 + rank], dtype=torch.float64)
    dist.all_reduce(tt, op=dist.ReduceOp.MAX)
    # result assembly is optional for a caller; used here only to check the shards
    dist.all_reduce(outs, op=dist.ReduceOp.SUM)
    if rank == 0:
        ret["units"] = units
        ret["t_max"] = float(tt.item())
        ret["out"] = outs.numpy()
    dist.destroy_process_group()


def test_two_ranks_cover_all_units_once_and_match_the_unsharded_oracle():
    from oracle import fasa_oracle as O

    for n in (1, 7, 8, 128):
        for world in (1, 2, 3, 8):
            got = sum((synth.shard_units(n, r, world) for r in range(world)), [])
            assert got == list(range(n))
            sizes = [len(synth.shard_units(n, r, world)) for r in range(world)]
            assert max(sizes) - min(sizes) <= 1
    port = _free_port()
    with mp.Manager() as m:
        ret = m.dict()
        mp.spawn(_rank_main, args=(2, port, ret), nprocs=2, join=True)
        ret = dict(ret)
    assert ret["t_max"] == 11.0
    w = synth.CONFIGS["c2"].replace(batch=3, n_q_heads=12, n_kv_heads=3, max_len=300, len_lo=100, len_hi=300, budget=32)
    t = synth.make_inputs(w, "cpu")
    full = O.decode_bf16(synth.bf16_bits(t["q"]), synth.bf16_bits(t["k"]), synth.bf16_bits(t["v"]), t["seq_lens"].numpy(),
                         t["dom"].numpy(), budget=w.budget, n_threads=2, want_dense=False)
    assert np.array_equal(ret["out"], full["out"])
