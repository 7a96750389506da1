"""GPU parity of the rotary embedding against the fp64 CPU checker, element by element, for
bf16 / fp16 / fp32, the vector and the element-wise kernel, small and very large positions."""
import numpy as np
import pytest
import torch

import oracle
import paper_2603_21331_b200 as ak
from paper_2603_21331_b200 import synth
from parity import assert_close_dt, guarded

pytestmark = pytest.mark.gpu
DEV = "cuda"
NAME = synth.DTYPE_NAMES
DTS = [torch.bfloat16, torch.float16, torch.float32]
ROUND = {torch.bfloat16: 2.0 ** -8 * 1.02, torch.float16: 2.0 ** -11 * 1.02, torch.float32: 2.0 ** -23}


def _assert_rope_close(y, ref, x, what):
    """The main bar of the element type, plus a one-rounding bound.  An output is a difference
    of two products and may cancel, so the fp32 evaluation error (cos / sin right to fp32
    rounding, two roundings in the multiply-add) is taken relative to |x0| + |x1| of the pair."""
    assert_close_dt(y, ref, what, tight=False)
    got = y.detach().cpu().double().numpy()
    xd = x.detach().cpu().double().numpy()
    mag = np.abs(xd[..., 0::2]) + np.abs(xd[..., 1::2])
    mag = np.repeat(mag, 2, axis=-1)
    bound = ROUND[y.dtype] * np.abs(ref) + 4e-7 * mag + 1e-37
    worst = float(np.max(np.abs(got - ref) / bound))
    assert worst <= 1.0, f"{what}: exceeds one-rounding bound by {worst:.3f}x"


SHAPES = [(64, 33, 128), (3, 17, 8), (1, 1, 2), (5, 7, 6), (4, 129, 96), (7, 5, 512), (9, 4, 64), (2, 300, 12),
          (130, 3, 128), (1, 2048, 128)]


@pytest.mark.parametrize("dtype", DTS)
@pytest.mark.parametrize("n_seq,S,Dh", SHAPES)
def test_rope_parity(n_seq, S, Dh, dtype):
    x = synth.rope_inputs(n_seq, S, Dh, synth.case_seed(18, n_seq * 131 + S * 7 + Dh), dtype=dtype)
    xd = x.to(DEV)
    for off in (0, 3, 100003):
        ref = oracle.rope(synth.to_elems(x), NAME[dtype], pos_offset=off)
        y, check = guarded((n_seq, S, Dh), dtype, DEV)
        ak.ak_rope_fwd(xd, y, pos_offset=off)
        torch.cuda.synchronize()
        check()
        _assert_rope_close(y, ref, x, f"rope {NAME[dtype]} {n_seq}x{S}x{Dh} offset {off}")
    # another base
    ref = oracle.rope(synth.to_elems(x), NAME[dtype], base=500000.0, pos_offset=1)
    _assert_rope_close(ak.ak_rope_fwd(xd, base=500000.0, pos_offset=1), ref, x, "rope base 5e5")


@pytest.mark.parametrize("dtype", DTS)
def test_rope_position_zero_is_the_identity_and_huge_positions_stay_exact(dtype):
    x = synth.rope_inputs(6, 1, 128, 1801, dtype=dtype)
    y = ak.ak_rope_fwd(x.to(DEV))
    assert torch.equal(y.cpu().view(torch.uint8), x.view(torch.uint8))        # cos 0 = 1, sin 0 = 0: bit copy
    # position ~1e9: an angle formed in fp32 would be off by tens of radians for pair 0
    x = synth.rope_inputs(3, 9, 64, 1802, dtype=dtype)
    for off in (10 ** 9, 2 ** 40 + 12345):
        ref = oracle.rope(synth.to_elems(x), NAME[dtype], pos_offset=off)
        _assert_rope_close(ak.ak_rope_fwd(x.to(DEV), pos_offset=off), ref, x, f"rope {NAME[dtype]} offset {off}")


@pytest.mark.parametrize("dtype", DTS)
def test_rope_misaligned_in_place_and_determinism(dtype):
    n_seq, S, Dh = 5, 19, 64
    x = synth.rope_inputs(n_seq, S, Dh, 1803, dtype=dtype)
    ref = oracle.rope(synth.to_elems(x), NAME[dtype], pos_offset=2)
    n = n_seq * S * Dh
    for xo, yo in ((1, 1), (0, 3), (2, 0), (0, 0)):
        xbuf = torch.zeros(n + 8, dtype=dtype, device=DEV)
        ybuf = torch.zeros(n + 8, dtype=dtype, device=DEV)
        xv, yv = xbuf[xo:xo + n].view(n_seq, S, Dh), ybuf[yo:yo + n].view(n_seq, S, Dh)
        xv.copy_(x)
        ak.ak_rope_fwd(xv, yv, pos_offset=2)
        torch.cuda.synchronize()
        _assert_rope_close(yv, ref, x, f"rope {NAME[dtype]} element offsets {xo},{yo}")
        assert bool((ybuf[:yo] == 0).all()) and bool((ybuf[yo + n:] == 0).all())
        # the element-wise kernel and the vector kernel agree bit for bit
        if (xo, yo) != (0, 0):
            assert torch.equal(yv.view(torch.uint8), ak.ak_rope_fwd(x.to(DEV), pos_offset=2).view(torch.uint8))
    xd = x.to(DEV)
    ak.ak_rope_fwd(xd, xd, pos_offset=2)
    _assert_rope_close(xd, ref, x, f"rope {NAME[dtype]} in place")
    big = synth.rope_inputs(64, 512, 128, 1804, device=DEV, dtype=dtype)
    first = ak.ak_rope_fwd(big).view(torch.uint8).clone()
    for _ in range(2):
        torch.empty(64 << 20, dtype=torch.uint8, device=DEV).fill_(1)
        assert torch.equal(first, ak.ak_rope_fwd(big).view(torch.uint8))
    e = torch.empty((0, 4, 8), dtype=dtype, device=DEV)
    assert ak.ak_rope_fwd(e).shape == (0, 4, 8)


def test_rope_adversarial_values():
    # large, tiny and mixed magnitudes: the rotation must neither overflow fp32 nor lose the small partner
    x = torch.zeros((2, 4, 8), dtype=torch.bfloat16)
    x[0, :, 0::2] = 65024.0
    x[0, :, 1::2] = -65024.0
    x[1, :, 0::2] = 1e-30
    x[1, :, 1::2] = 3.0
    for dtype in (torch.bfloat16, torch.float32):
        xx = x.to(dtype)
        ref = oracle.rope(synth.to_elems(xx), NAME[dtype], pos_offset=5)
        y = ak.ak_rope_fwd(xx.to(DEV), pos_offset=5)
        assert torch.isfinite(y.float()).all()
        _assert_rope_close(y, ref, xx, f"rope adversarial {NAME[dtype]}")
