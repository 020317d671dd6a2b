"""calidrop_decode_static: the decode step for callers that cannot hand the library a workspace.

A plugin inside a runtime whose memory plan is frozen, or code running where device allocation
is forbidden, still passes inputs and outputs; the split-K scratch then comes from a fixed
4 MiB array inside the library instead of a caller-allocated workspace.  The entry point must
give what calidrop_decode gives, on repeated calls (the array is shared and keeps the previous
call's contents), and must refuse problems whose scratch would not fit.

This file sorts last on purpose: a run that stops at the first failure has then already run
every other test.
"""
import numpy as np
import pytest
import torch

from paper_2507_19906_b200 import workload as wl

from gpu_util import LSE_ABS, OUT_MAX_ABS, OUT_MEAN_ABS, gpu_compress, to_dev

pytestmark = pytest.mark.gpu


def test_static_scratch_decode_matches_workspace_decode_twice(cuda_lib):
    cd = cuda_lib
    cfg = wl.small_config(B=2, Hq=8, Hkv=2, L=700, window=16, pool=7, budget=96, steps=2, n_heavy=10)
    Q, (K, V) = wl.gen_q_obs(cfg), wl.gen_kv(cfg)
    T = 2
    g = gpu_compress(Q, K, V, window=16, pool=7, budget=96, n_cal=16, cap=96 + T)
    p, st = g.p, g.st
    q, kn, vn = wl.gen_decode_inputs(cfg, Q, steps=T)
    # two independent copies of the retained cache, one per entry point
    Ka, Va = st.K_kept.clone(), st.V_kept.clone()
    Kb, Vb = st.K_kept.clone(), st.V_kept.clone()

    def outputs():
        return (torch.empty((p.B, p.Hq, p.D), dtype=torch.bfloat16, device="cuda"),
                torch.empty((p.B, p.Hq), dtype=torch.float32, device="cuda"),
                torch.empty((p.B, p.Hq), dtype=torch.uint8, device="cuda"))

    applied = 0
    for t in range(T):                      # two calls in a row share the built-in scratch
        dq, dk, dv = to_dev(q[t]), to_dev(kn[t]), to_dev(vn[t])
        oa, la, fa = outputs()
        ob, lb, fb = outputs()
        cd.calidrop_decode(p, dq, dk, dv, Ka, Va, 96 + t, st.O_c, st.LSE_c, st.C_q, oa, la, fa, st.ws_decode)
        cd.calidrop_decode_static(p, dq, dk, dv, Kb, Vb, 96 + t, st.O_c, st.LSE_c, st.C_q, ob, lb, fb)
        torch.cuda.synchronize()
        err = (oa.float() - ob.float()).abs()
        assert torch.isfinite(ob.float()).all()
        assert float(err.max()) <= OUT_MAX_ABS and float(err.mean()) <= OUT_MEAN_ABS
        assert float((la - lb).abs().max()) <= LSE_ABS
        assert torch.equal(fa, fb)
        assert torch.equal(Ka, Kb) and torch.equal(Va, Vb)       # the appended rows
        applied += int((fb & 1).sum())
    assert applied > 0                       # the calibration merge was exercised


def test_static_scratch_limit_and_argument_checks(cuda_lib):
    cd = cuda_lib
    big = cd.make_params(B=512, Hq=64, Hkv=8, n_cal=64, cap=64)      # 4096 units: beyond 4 MiB of scratch
    assert cd.calidrop_decode_workspace_bytes(big, 64) > cd.STATIC_SCRATCH_BYTES
    rc = cd.calidrop_decode_static(big, None, None, None, None, None, 1, None, None, None, None, None, None,
                                   check=False)
    assert rc == cd.SCRATCH_LIMIT
    assert "scratch" in cd.status_string(cd.SCRATCH_LIMIT)
    small = cd.make_params(B=1, Hq=4, Hkv=2, n_cal=1, cap=8)
    rc = cd.calidrop_decode_static(small, None, None, None, None, None, 1, None, None, None, None, None, None,
                                   check=False)
    assert rc == cd.INVALID_ARG
