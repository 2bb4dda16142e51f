"""bitlinear_quant_act_noalloc against bitlinear_quant_act.

Some callers of this library may not allocate device memory at the moment they call it: a plug-in
running inside another framework's stream callback, a real-time loop with a fixed memory budget, a
binding that only forwards the pointers it was handed.  For them the library keeps the per-tensor
statistics of LN + quantisation in a fixed array of its own.  The entry point runs the same kernels
as bitlinear_quant_act, so its outputs must be bit-identical to it - on the first call and on a
second one that follows immediately with other data (the array keeps the first call's contents) -
and, like every quantising entry point, within the stated bars of the CPU oracle.

This file is named so that pytest collects it after every other test file.
"""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2310_11453_b200 import binding as B
from paper_2310_11453_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _outputs(M, K, G, gran):
    ns = (M, G) if gran == B.PER_TOKEN else (G,)
    return dict(x_q=torch.full((M, K), 99, dtype=torch.int8, device=DEV),
                gamma=torch.full(ns, -1.0, dtype=torch.float32, device=DEV),
                eta=torch.full(ns, -1.0, dtype=torch.float32, device=DEV))


def _same(a, b):
    return all(torch.equal(a[k], b[k]) for k in ("x_q", "gamma", "eta"))


@pytest.mark.parametrize("mode,gran,G", [(B.ABSMAX, B.PER_TENSOR, 1), (B.ETA, B.PER_TENSOR, 4),
                                         (B.ABSMAX, B.PER_TOKEN, 2)])
def test_two_calls_in_a_row_match_the_workspace_entry_point(mode, gran, G):
    K = 1024
    # two different problems, the second larger in M than the first, back to back on one stream
    cases = [(96, 11), (200, 12)]
    xs = [synth.make_x(M, K, torch.bfloat16, seed=seed, outliers=(mode == B.ABSMAX),
                       relu=(mode == B.ETA)).to(DEV) for M, seed in cases]
    got = [_outputs(x.shape[0], K, G, gran) for x in xs]
    for x, out in zip(xs, got):                       # nothing between the two calls
        B.quant_act_noalloc(x, G=G, mode=mode, gran=gran, out=out)
    assert B.noalloc_status() == B.OK                 # synchronises; no bounded wait of the calls ran out
    for x, out in zip(xs, got):
        ref = B.quant_act(x, G=G, mode=mode, gran=gran, out=_outputs(x.shape[0], K, G, gran))
        torch.cuda.synchronize()
        assert _same(out, ref)
        assert out["x_q"].abs().max().item() <= 127
        # and against the CPU oracle, at the bars of the other quantisation tests: codes +-1 on at most
        # 1e-4 of the elements, gamma and eta to 2e-6 relative
        want = O.quant_act(x.float().cpu().numpy(), G=G, mode=mode, gran=gran, ln_eps=1e-5)
        diff = out["x_q"].cpu().numpy().astype(np.int32) - want["codes"].astype(np.int32)
        assert np.abs(diff).max() <= 1 and np.count_nonzero(diff) <= max(1, int(1e-4 * diff.size))
        np.testing.assert_allclose(out["gamma"].cpu().numpy(), want["gamma"], rtol=2e-6)
        if mode == B.ETA:
            np.testing.assert_allclose(out["eta"].cpu().numpy(), want["eta"], rtol=2e-6, atol=1e-6)


def test_sizes_beyond_the_built_in_scratch_are_refused():
    K = 64
    M = B.NOALLOC_MAX_SEGMENTS + 1
    x = torch.zeros((M, K), dtype=torch.float32, device=DEV)
    out = _outputs(M, K, 1, B.PER_TENSOR)
    with pytest.raises(B.BitLinearError) as err:
        B.quant_act_noalloc(x, gran=B.PER_TENSOR, out=out)
    assert err.value.code == B.ERR_TOO_LARGE
    torch.cuda.synchronize()
    assert (out["x_q"] == 99).all()                   # nothing was launched
    # the same size is fine per token (no scratch involved), and at the limit per tensor
    B.quant_act_noalloc(x, gran=B.PER_TOKEN, out=_outputs(M, K, 1, B.PER_TOKEN))
    xl = x[: B.NOALLOC_MAX_SEGMENTS]
    B.quant_act_noalloc(xl, gran=B.PER_TENSOR, out=_outputs(xl.shape[0], K, 1, B.PER_TENSOR))
    torch.cuda.synchronize()
