"""The allocation-free predictor entry point gives the oracle's (and np_predict's) logits.

Collected last on purpose (file name): a failure here cannot hide the result of
any other test in a run that stops at the first failure.
"""
import numpy as np
import pytest
import torch

from paper_2608_22643_b200 import binding as nb
from paper_2608_22643_b200 import build as nbuild
from paper_2608_22643_b200 import synth
from oracle import np_oracle as O
from tests.harness import Pair, rel_l2, u16

pytestmark = pytest.mark.gpu


_WIDE = synth.StackConfig("noalloc_wide", 2, 256, 1024 + 32, 2048, 10, 20, 4, 13, 0.9)   # B = 1 takes the ring kernel
_FULL = synth.StackConfig("noalloc_full", 2, 512, 2048 + 32, 1024, 10, 20, 4, 17, 0.9)   # 16 x 1024 = the whole scratch


@pytest.mark.parametrize("cfg,B", [(synth.CONFIGS["small"], 1), (synth.CONFIGS["small"], 3), (_WIDE, 1), (_FULL, 16)])
def test_noalloc_predictor_matches_context_path_twice(cfg, B):
    """Callers that cannot allocate device memory (pool-owned memory, allocation-free decode
    loops) use np_predict_logits_noalloc; two calls in a row on the library's fixed scratch
    must both reproduce the oracle's predictor within tolerance and, bit for bit, what
    np_predict computes with its workspace on the same plain-core kernels."""
    p = Pair(cfg, max_batch=B, with_oracle=False, flags=nb.NP_F_CHECK_BOUNDS | nb.NP_F_NO_TENSOR_CORES)
    try:
        L, M, D, H = cfg.n_layers, cfg.d_ffn, cfg.d_model, cfg.d_pred
        xs = synth.hidden_states(cfg, 2, batch=B)
        want = torch.empty((B, L, M), dtype=torch.float32, device="cuda")
        got = torch.full((B, L, M), float("nan"), dtype=torch.float32, device="cuda")
        for t in range(2):                                  # second call reuses the scratch
            x = xs[t].cuda()
            nb.np_predict(p.eng.ctx, x, B, want, None, p.eng.stream)
            p.eng.stream.synchronize()
            nb.np_predict_logits_noalloc(p.eng.w1, p.eng.w2, x, B, L, D, M, H, got, p.eng.stream)
            assert nb.np_noalloc_check(p.eng.stream) == nb.NP_OK      # no bounded wait ran out
            z = O.predict(u16(p.w1_cpu), u16(p.w2_cpu), u16(xs[t]), L, M)
            assert rel_l2(got.cpu().numpy(), z) < 1e-5
            assert np.isfinite(got.cpu().numpy()).all()
            assert torch.equal(got, want)
            got.fill_(float("nan"))
    finally:
        p.close()


def test_noalloc_rejects_oversize_and_bad_arguments():
    nbuild.build()
    lib = nb.load()
    z = torch.zeros(64, device="cuda")
    # B * d_pred above the fixed scratch (16 * 2048 > 16384 floats); nothing is launched
    rc = lib.np_predict_logits_noalloc(z.data_ptr(), z.data_ptr(), z.data_ptr(), 16, 1, 256, 1024, 2048,
                                       z.data_ptr(), None)
    assert rc == nb.NP_E_INVAL and "exceeds the fixed scratch" in lib.np_noalloc_last_error().decode()
    # a shape the library does not support at all
    rc = lib.np_predict_logits_noalloc(z.data_ptr(), z.data_ptr(), z.data_ptr(), 1, 2, 4096, 1024, 4096 + 8,
                                       z.data_ptr(), None)
    assert rc == nb.NP_E_INVAL
    ok_shape = (1, 1, 256, 1024, 64)
    assert lib.np_predict_logits_noalloc(None, z.data_ptr(), z.data_ptr(), *ok_shape, z.data_ptr(), None) == nb.NP_E_INVAL
    assert lib.np_predict_logits_noalloc(z.data_ptr() + 4, z.data_ptr(), z.data_ptr(), *ok_shape, z.data_ptr(), None) == nb.NP_E_INVAL
    assert lib.np_noalloc_last_error().decode()
    with pytest.raises(nb.NpError) as e:
        nb.np_predict_logits_noalloc(z, z, z, 9, 1, 256, 1024, 2048, z)
    assert "exceeds the fixed scratch" in str(e.value)
