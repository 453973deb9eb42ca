"""Parity of the DCN cross layer (forward partials + aggregate, backward) against the CPU oracle.
Needs a B200."""
import numpy as np
import pytest
import torch

import oracle

pytestmark = pytest.mark.gpu


def _close(got, ref, what, extra=None):
    tol = 1e-5 * np.abs(ref) + 1e-6 + (0 if extra is None else extra)
    bad = np.abs(got.astype(np.float64) - ref) > tol
    assert not bad.any(), (what, int(bad.sum()), float(np.abs(got - ref).max()))


@pytest.mark.parametrize("B,d,S", [(1, 1, 1), (7, 23, 3), (300, 1248, 16), (2048, 4099, 64), (64, 64, 64)])
def test_cross_layer_parity(B, d, S):
    from paper_1909_04823_b200 import binding
    rng = np.random.default_rng([B, d, S])
    x0, x, gY = (rng.standard_normal((B, d)).astype(np.float32) for _ in range(3))
    w = (rng.standard_normal(d) / np.sqrt(d)).astype(np.float32)
    b = rng.standard_normal(d).astype(np.float32)
    dev = lambda a: torch.from_numpy(a).cuda()
    y, P, part = binding.cross_forward(dev(x0), dev(x), dev(w), dev(b), S, want_part=True)
    torch.cuda.synchronize()
    ref = oracle.cross_forward(x0, x, w, b, S)
    sum_tol = 2e-6 * ref["Sabs"]                       # float32 dot products: error against the size of the terms
    _close(part.cpu().numpy(), ref["part"], "part", extra=sum_tol[None])
    _close(P.cpu().numpy(), ref["P"], "P", extra=sum_tol)
    _close(y.cpu().numpy(), ref["y"], "y", extra=(np.abs(x0) * sum_tol[:, None]))
    # backward from the oracle's aggregate (stage-wise: forward differences do not leak in)
    P32 = ref["P"].astype(np.float32)
    gx0, gx, gw, gb = binding.cross_backward(dev(x0), dev(x), dev(w), dev(P32), dev(gY))
    torch.cuda.synchronize()
    rb = oracle.cross_backward(x0, x, w, P32, gY)
    t_tol = 2e-6 * np.sum(np.abs(gY.astype(np.float64) * x0), axis=1)
    _close(gx0.cpu().numpy(), rb["gx0"], "gx0")
    _close(gx.cpu().numpy(), rb["gx"], "gx", extra=np.abs(w)[None] * t_tol[:, None])
    tx = np.abs(rb["t"])[:, None] * np.abs(x)
    _close(gw.cpu().numpy(), rb["gw"], "gw", extra=2e-6 * tx.sum(0) + (t_tol[:, None] * np.abs(x)).sum(0))
    _close(gb.cpu().numpy(), rb["gb"], "gb", extra=2e-6 * np.abs(gY).sum(0))


def test_cross_layer_rejects_bad_arguments_and_is_deterministic():
    from paper_1909_04823_b200 import binding
    x = torch.randn(32, 40, device="cuda")
    w = torch.randn(40, device="cuda")
    with pytest.raises(binding.DesError):
        binding.cross_forward(x, x, w, w, 41)           # more shards than columns
    y, P, _ = binding.cross_forward(x, x, w, w, 5)
    outs = [binding.cross_backward(x, x, w, P, y) for _ in range(3)]
    torch.cuda.synchronize()
    for o in outs[1:]:
        for a, c in zip(o, outs[0]):
            assert torch.equal(a, c)
