"""The one exchange step of batch-sharded channel-wise quantization, on CPU with two gloo ranks: each
rank holds half of the batch, the ranges are all-reduced, and quantizing each half with the reduced
range must give exactly the halves of what the oracle gives on the whole batch."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _case():
    rng = np.random.default_rng(21)
    x = (rng.standard_normal((8, 6, 5, 5)) * np.exp(rng.standard_normal((1, 6, 1, 1)))).astype(np.float32)
    x[:4, 2] = np.maximum(x[:4, 2], 0)          # channel 2: the minimum lives in the second half only
    x[4:, 3] = 0.0                              # channel 3: all-zero on rank 1, so its local range is degenerate
    x[:, 4] = np.maximum(x[:, 4], 0)            # channel 4: post-ReLU everywhere, the global minimum is +0
    gy = rng.standard_normal(x.shape).astype(np.float32)
    return x + np.float32(0), gy


def _rank(rank: int, world: int, port: int, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from oracle import granq_oracle as orc
    from paper_2503_18339_b200.data_parallel import sync_range
    x, gy = _case()
    n = x.shape[0] // world
    xs, gs = x[rank * n:(rank + 1) * n], gy[rank * n:(rank + 1) * n]
    lo, hi = orc.range_(xs)                                        # Eq. 4 on this rank's slice
    tlo, thi = torch.from_numpy(lo.copy()), torch.from_numpy(hi.copy())
    sync_range(tlo, thi)                                           # the exchange
    res = orc.fakequant(xs, 3, tlo.numpy(), thi.numpy(), gy=gs)    # Eq. 5, 1, 6, STE with the global range
    out[rank] = (lo, hi, tlo.numpy().copy(), thi.numpy().copy(), res.y, res.gx, res.codes)
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_quantize_with_the_range_of_the_whole_batch():
    from oracle import granq_oracle as orc
    world, port = 2, 31500 + os.getpid() % 2000
    out = mp.get_context("spawn").Manager().dict()
    mp.spawn(_rank, args=(world, port, out), nprocs=world, join=True)
    x, gy = _case()
    ref = orc.fused(x, 3, gy=gy)
    bits = lambda a: np.ascontiguousarray(a).view(np.uint32)       # noqa: E731
    for r in range(world):
        lo_local, hi_local, lo, hi, y, gx, codes = out[r]
        assert np.array_equal(bits(lo), bits(ref.lo)) and np.array_equal(bits(hi), bits(ref.hi))
        half = slice(r * 4, (r + 1) * 4)
        assert np.array_equal(bits(y), bits(ref.y[half])) and np.array_equal(bits(gx), bits(ref.gx[half]))
        assert np.array_equal(codes, ref.codes[half])
    # the exchange mattered: the local ranges differ from the global one on both ranks
    assert not np.array_equal(out[0][0], ref.lo) and not np.array_equal(out[1][1], ref.hi)
    for r in range(world):                                          # a zero minimum stays +0 through the exchange
        assert out[r][2][4] == 0 and not np.signbit(out[r][2][4])


def test_sync_range_is_a_no_op_without_a_process_group():
    sys.path.insert(0, ROOT)
    from paper_2503_18339_b200.data_parallel import sync_range
    lo, hi = torch.tensor([0.0, -1.0]), torch.tensor([2.0, 3.0])
    sync_range(lo, hi)
    assert lo.tolist() == [0.0, -1.0] and hi.tolist() == [2.0, 3.0]
