"""Data parallelism, the parts that need no GPU: the shard map (host arithmetic in the library) and,
with two gloo ranks on CPU, the exchange step around it -- reduce-scatter of the gradients, the update
of each rank's shard, all-gather of the compute copies -- against the oracle's AdamW on the summed
gradients of the whole model."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import fax_oracle as O
from paper_2204_06514_b200 import build, dp

HP = dict(lr=1e-3, beta1=0.9, beta2=0.95, eps=1e-8)
SIZES = [50304 * 8, 1024 * 8, 8, 8, 8 * 24, 24, 64, 8, 1, 129, 4096, 7]     # ragged on purpose


@pytest.fixture(scope="module", autouse=True)
def _lib():
    build.build()


@pytest.mark.parametrize("world", [1, 2, 3, 8])
@pytest.mark.parametrize("sizes", [SIZES, [1], [128, 128], [5, 1000003, 3]])
def test_shard_map_covers_every_element_once(world, sizes):
    align = dp.ALIGN
    offsets, total = dp.layout(sizes, world)
    assert total % (align * world) == 0 and all(o % align == 0 for o in offsets)
    for i in range(len(sizes) - 1):
        assert offsets[i] + sizes[i] <= offsets[i + 1] < offsets[i] + sizes[i] + align
    assert total >= offsets[-1] + sizes[-1]
    owner = [np.full(n, -1, np.int32) for n in sizes]
    for rank in range(world):
        lo, ln, pieces = dp.shard_map(sizes, world, rank)
        assert ln == total // world and lo == rank * ln and ln % align == 0
        for t, b, e, fb in pieces:
            assert 0 <= b < e <= sizes[t]
            assert fb == offsets[t] + b and lo <= fb and fb + (e - b) <= lo + ln
            assert b == 0 or fb == lo                 # a piece starts at a tensor's start or at the shard's
            assert np.all(owner[t][b:e] == -1)
            owner[t][b:e] = rank
    assert all(np.all(o >= 0) for o in owner)


def test_shard_map_rejects_bad_arguments():
    from paper_2204_06514_b200 import binding as fx
    for kw in (dict(world=0, rank=0), dict(world=2, rank=2), dict(world=2, rank=-1)):
        with pytest.raises(fx.FaxError) as e:
            dp.shard_map([10, 20], kw["world"], kw["rank"])
        assert e.value.status == fx.FAX_ERR_INVALID_ARG
    with pytest.raises(fx.FaxError):
        dp.layout([10], 1, align=24)                   # not a power of two


def _rank_grads(rank, sizes):
    rng = np.random.default_rng(100 + rank)
    return [(rng.standard_normal(n) * 10.0 ** rng.uniform(-6, 0, n)).astype(np.float32) for n in sizes]


def _weights(sizes):
    rng = np.random.default_rng(7)
    return [rng.standard_normal(n).astype(np.float32) for n in sizes]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    sizes = SIZES
    offsets, total = dp.layout(sizes, world)
    lo, ln, pieces = dp.shard_map(sizes, world, rank)
    w = torch.zeros(total, dtype=torch.float64)
    g = torch.zeros(total, dtype=torch.float32)
    for off, n, a, gr in zip(offsets, sizes, _weights(sizes), _rank_grads(rank, sizes)):
        w[off:off + n] = torch.as_tensor(a, dtype=torch.float64)
        g[off:off + n] = torch.as_tensor(gr) / world          # each rank's share of the mean
    g_shard = torch.zeros(ln, dtype=torch.float32)
    dp.reduce_scatter_sum(g, g_shard, rank, world)
    wc = torch.zeros(total, dtype=torch.float32)               # stands for the compute copy that is gathered
    for t, b, e, fb in pieces:                                 # the update of this rank's pieces
        nw, _, _ = O.adamw(w[fb:fb + e - b].numpy(), 0.0, 0.0, g_shard[fb - lo:fb - lo + e - b].numpy(),
                           weight_decay=0.1, step=1, **HP)
        wc[fb:fb + e - b] = torch.as_tensor(nw, dtype=torch.float32)
    dp.all_gather_shards(wc, rank, world)
    out[rank] = wc.numpy().copy()
    dist.barrier()
    dist.destroy_process_group()


def test_sharded_update_equals_adamw_on_the_summed_gradients_world2():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    world = 2
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        got0, got1 = out[0], out[1]
    assert np.array_equal(got0, got1)                          # every rank ends with the same weights
    offsets, _ = dp.layout(SIZES, world)
    grads = [_rank_grads(r, SIZES) for r in range(world)]
    for i, (off, n, a) in enumerate(zip(offsets, SIZES, _weights(SIZES))):
        gsum = sum((grads[r][i] / np.float32(world)).astype(np.float32) for r in range(world))
        ref, _, _ = O.adamw(a.astype(np.float64), 0.0, 0.0, gsum, weight_decay=0.1, step=1, **HP)
        assert np.allclose(got0[off:off + n], ref, rtol=0, atol=2e-7 * max(1.0, np.abs(ref).max())), i
