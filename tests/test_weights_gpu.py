"""GPU parity of the batched channel-wise weight fake-quantization (Section 5.1) against the CPU
oracle: one launch over all weight tensors of a network must give, tensor by tensor, exactly what
the oracle's fused path gives with channel_axis = 0 (lo / hi / s / z / y / gx bit for bit)."""
import numpy as np
import pytest
import torch

from oracle import granq_oracle as orc
from paper_2503_18339_b200 import workloads as wl
from test_parity_gpu import b, same_bits, to_dev, to_np  # noqa: F401

pytestmark = pytest.mark.gpu


def as4d(w: np.ndarray) -> np.ndarray:
    return w.reshape(w.shape[0], -1, 1, 1) if w.ndim != 4 else w


def check_batch(b, ws, gs, bits, dtype):
    if dtype == "bf16":
        ws = [wl.to_bf16_bits(w) for w in ws]
        gs = None if gs is None else [wl.to_bf16_bits(g) for g in gs]
    outs = b.granq_fakequant_weights([to_dev(w) for w in ws], bits, grads=None if gs is None else [to_dev(g) for g in gs],
                                     want_params=True)
    torch.cuda.synchronize()
    for i, (w, o) in enumerate(zip(ws, outs)):
        bi = bits if isinstance(bits, int) else bits[i]
        ref = orc.fused(as4d(w), bi, gy=None if gs is None else as4d(gs[i]), channel_axis=0)
        assert same_bits(to_np(o.lo), ref.lo) and same_bits(to_np(o.hi), ref.hi), f"range of tensor {i}"
        assert same_bits(to_np(o.s), ref.s) and same_bits(to_np(o.z), ref.z), f"parameters of tensor {i}"
        y = to_np(o.y).reshape(ref.y.shape)
        tol = 1e-6 * ref.s.astype(np.float64).reshape(-1, 1, 1, 1)
        wide = (lambda a: wl.bf16_bits_to_f32(a) if a.dtype == np.uint16 else a)
        assert np.all(np.abs(wide(y).astype(np.float64) - wide(ref.y).astype(np.float64)) <= tol)
        assert same_bits(y, ref.y), f"y of tensor {i}"
        if gs is not None:
            assert same_bits(to_np(o.gx).reshape(ref.gx.shape), ref.gx), f"gx of tensor {i}"


@pytest.mark.parametrize("net", ["resnet20", "resnet18"])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_all_weights_of_a_network_in_one_launch(b, net, dtype):
    ws, gs = wl.make_weights(net), wl.make_weights(net, grads=True)
    check_batch(b, ws, gs, 4, dtype)
    check_batch(b, ws, None, [3 + i % 3 for i in range(len(ws))], dtype)      # forward only, mixed bit-widths


def test_odd_shapes_constant_channels_and_one_tensor(b):
    rng = np.random.default_rng(3)
    ws = [rng.standard_normal(s).astype(np.float32) for s in [(5, 27), (1, 1), (7, 3, 3, 3), (4, 1024), (3, 4100), (2, 8)]]
    ws[3][1] = 0.0                       # an all-zero channel
    ws[3][2] = -2.5                      # a constant channel
    ws[5][0, :3] = [-3.5, -2.0, -1.0]    # ties
    gs = [rng.standard_normal(w.shape).astype(np.float32) for w in ws]
    for bits in (2, 8):
        check_batch(b, ws, gs, bits, "f32")
    check_batch(b, ws[:1], gs[:1], 3, "f32")
    # unaligned base pointer: the scalar path
    base = to_dev(np.concatenate([np.zeros(1, np.float32), ws[3].ravel()]))
    out = b.granq_fakequant_weights([base[1:].view(4, 1024)], 4, want_params=True)[0]
    ref = orc.fused(as4d(ws[3]), 4, channel_axis=0)
    assert same_bits(to_np(out.y).reshape(ref.y.shape), ref.y) and same_bits(to_np(out.lo), ref.lo)


def test_weights_reject_bad_arguments(b):
    w = to_dev(np.ones((4, 8), np.float32))
    with pytest.raises(b.GranqError) as err:
        b.granq_fakequant_weights([w], 9)
    assert err.value.status == b.ERR_INVALID_ARG
    with pytest.raises(b.GranqError) as err:
        b.granq_fakequant_weights([w], 4, workspace=torch.empty(16, dtype=torch.uint8, device="cuda"))
    assert err.value.status == b.ERR_WORKSPACE
