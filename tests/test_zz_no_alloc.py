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


def test_static_scratch_carries_the_partials_of_a_unit_split_over_clusters(cuda_lib):
    """One unit with 17000 cached rows: the unit is split over two clusters, whose partial results,
    arrival counter and error word all live in the built-in array.  Two calls in a row on the shared
    array, each checked against the workspace entry point and against the oracle; the device's free
    memory must not move (nothing is allocated or freed by the calls)."""
    import oracle
    from gpu_util import assert_close_lse, assert_close_out, to_bits
    cd = cuda_lib
    rng = np.random.Generator(np.random.Philox(key=[93, 7]))
    B, Hq, Hkv, D, kv0, n_cal = 1, 4, 1, 128, 17000, 2
    cap = kv0 + 2
    bits = lambda x: wl.f32_to_bf16_bits(np.ascontiguousarray(x, dtype=np.float32))
    p = cd.make_params(B=B, Hq=Hq, Hkv=Hkv, L=kv0 + 64, window=8, pool=7, budget=kv0, n_cal=n_cal, cap=cap)
    p.theta1, p.theta2 = 0.7, -1.0
    assert cd.calidrop_decode_workspace_bytes(p, cap) <= cd.STATIC_SCRATCH_BYTES
    Kk = np.zeros((B, Hkv, cap, D), dtype=np.uint16); Vk = np.zeros_like(Kk)
    Kk[:, :, :kv0] = bits(rng.standard_normal((B, Hkv, kv0, D)))
    Vk[:, :, :kv0] = bits(rng.standard_normal((B, Hkv, kv0, D)))
    Cq = bits(rng.standard_normal((B, Hq, n_cal, D)))
    Oc = rng.standard_normal((B, Hq, n_cal, D)).astype(np.float32)
    Lc = (rng.standard_normal((B, Hq, n_cal)) + 9.0).astype(np.float32)
    Ka, Va, Kb, Vb = to_dev(Kk), to_dev(Vk), to_dev(Kk), to_dev(Vk)
    dCq, dOc, dLc = to_dev(Cq), torch.from_numpy(Oc).cuda(), torch.from_numpy(Lc).cuda()
    ws = torch.zeros((cd.calidrop_decode_workspace_bytes(p, cap),), dtype=torch.uint8, device="cuda")
    outs = [(torch.empty((B, Hq, D), dtype=torch.bfloat16, device="cuda"),
             torch.empty((B, Hq), dtype=torch.float32, device="cuda"),
             torch.empty((B, Hq), dtype=torch.uint8, device="cuda")) for _ in range(2)]
    steps = []
    for t in range(2):
        q = bits(wl.bf16_bits_to_f32(Cq[:, :, t % n_cal]) + 0.5 * rng.standard_normal((B, Hq, D)).astype(np.float32))
        steps.append((q, bits(rng.standard_normal((B, Hkv, D))), bits(rng.standard_normal((B, Hkv, D)))))
    dev_steps = [(to_dev(q), to_dev(kn), to_dev(vn)) for q, kn, vn in steps]
    # first call on this device outside the measured window (it resolves the array's address once)
    (oa, la, fa), (ob, lb, fb) = outs
    torch.cuda.synchronize()
    free_before = None
    for t, ((q, kn, vn), (dq, dk, dv)) in enumerate(zip(steps, dev_steps)):
        cd.calidrop_decode(p, dq, dk, dv, Ka, Va, kv0 + t, dOc, dLc, dCq, oa, la, fa, ws)
        cd.calidrop_decode_static(p, dq, dk, dv, Kb, Vb, kv0 + t, dOc, dLc, dCq, ob, lb, fb)
        torch.cuda.synchronize()
        if free_before is None:
            free_before = torch.cuda.mem_get_info()[0]
        o = oracle.decode(q, kn, vn, Kk, Vk, kv0 + t, Oc, Lc, Cq, theta1=0.7, theta2=-1.0)
        assert np.array_equal(fb.cpu().numpy() >> 2, o.flags >> 2)
        assert_close_out(wl.bf16_bits_to_f64(to_bits(ob)), o.out, f"static entry, step {t}")
        assert_close_lse(lb.cpu().numpy(), o.lse, f"static entry, step {t} lse")
        err = (oa.float() - ob.float()).abs()
        assert float(err.max()) <= OUT_MAX_ABS and float((la - lb).abs().max()) <= LSE_ABS
        assert torch.equal(fa, fb) and torch.equal(Ka, Kb) and torch.equal(Va, Vb)
    assert torch.cuda.mem_get_info()[0] == free_before       # the second call allocated and freed nothing


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
