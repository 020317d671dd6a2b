"""GPU parity: the CUDA path through the C-ABI against the fp64 oracle, element by element.

Tolerances: kept-index sets bit-exact except near-tie swaps
(oracle pooled votes within 1e-5 relative); K_kept/V_kept/C_q bit-exact; O_c and decode
outputs within max-abs 2e-2 and mean-abs 2e-3; LSE_c and the output LSE within 1e-3.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2507_19906_b200 import workload as wl

from gpu_util import (assert_close_lse, assert_close_out, compare_compress, decode_steps_compare,
                      gpu_compress, to_bits, to_dev)

pytestmark = pytest.mark.gpu


def _inputs(cfg, layer=0):
    Q = wl.gen_q_obs(cfg, layer)
    K, V = wl.gen_kv(cfg, layer)
    return Q, K, V


# ---------------------------------------------------------------- small shapes, every step
SMALL = [
    # B, Hq, Hkv, L, W, pool, budget, n_cal
    (1, 1, 1, 140, 1, 1, 9, 1),          # single window row, no pooling
    (1, 4, 2, 300, 8, 5, 40, 1),         # Algorithm 1 as printed (last query only)
    (2, 8, 2, 517, 16, 7, 100, 16),      # ragged L, G = 4, every window row calibrates
    (1, 7, 1, 1000, 32, 7, 128, 5),      # G = 7
    (1, 8, 1, 259, 4, 3, 30, 2),         # G = 8
    (2, 6, 3, 1301, 32, 5, 64, 32),      # spans several 128-key tiles with a ragged tail
    (1, 4, 4, 130, 64, 7, 65, 64),       # L - W < one tile, k_sel = 1
    (1, 2, 1, 96, 8, 7, 95, 3),          # a single evicted candidate
    (1, 7, 1, 700, 64, 7, 160, 64),      # 448 window rows per kv head: two row blocks in the vote pass
    (1, 16, 2, 900, 64, 5, 200, 16),     # G = 8, W = 64: 512 window rows, four 128-row statistic blocks
    (1, 4, 1, 3000, 128, 7, 400, 128),   # W = 128: one query head per calibration row block
    (1, 8, 1, 4000, 16, 7, 2100, 16),    # one unit: one cluster of eight CTAs, 263 rows each
    (2, 8, 2, 2500, 16, 7, 1000, 7),     # four units: most CTAs without a C_q row
    (1, 8, 1, 1500, 128, 7, 400, 4),     # 1024 window rows per kv head: the CUDA-core scoring and calibration kernels
    (1, 2, 1, 1200, 160, 5, 400, 160),   # window of 160 rows (beyond the 128-row tiles): the same kernels, n_cal = W
]


@pytest.mark.parametrize("B,Hq,Hkv,L,W,pool,budget,n_cal", SMALL)
def test_compress_and_decode_small(cuda_lib, B, Hq, Hkv, L, W, pool, budget, n_cal):
    cfg = wl.small_config(B=B, Hq=Hq, Hkv=Hkv, L=L, window=W, pool=pool, budget=budget, steps=5,
                          n_sink=2, n_heavy=max(1, L // 50))
    Q, K, V = _inputs(cfg)
    T = 5
    g = gpu_compress(Q, K, V, window=W, pool=pool, budget=budget, n_cal=n_cal, cap=budget + T)
    orc = oracle.compress(Q, K, V, window=W, pool=pool, budget=budget, n_cal=n_cal, cap=budget + T)
    # intermediate arrays, for a sharper diagnosis than the kept set alone
    np.testing.assert_allclose(g.row_lse, orc.row_lse, atol=2e-5)
    np.testing.assert_allclose(g.vote, orc.vote, rtol=2e-5, atol=1e-9)
    np.testing.assert_allclose(g.pooled, orc.pooled, rtol=2e-5, atol=1e-9)
    ref, _ = compare_compress(g, Q, K, V, window=W, pool=pool, budget=budget, n_cal=n_cal, orc=orc)
    q, kn, vn = wl.gen_decode_inputs(cfg, Q, steps=T)
    st = decode_steps_compare(g, ref, q, kn, vn, steps=T)
    assert st["total"] == T * B * Hq


def test_single_cta_selection_for_very_long_prompts(cuda_lib):
    """Beyond 262144 tokens the eight-CTA cluster selection no longer holds a unit's keys in registers
    and the single-CTA radix selection takes over; everything else is the usual path."""
    L, W, pool, budget, n_cal = 263000, 8, 7, 1000, 2
    cfg = wl.small_config(B=1, Hq=1, Hkv=1, L=L, window=W, pool=pool, budget=budget, steps=2, n_sink=4, n_heavy=300)
    Q, K, V = _inputs(cfg)
    g = gpu_compress(Q, K, V, window=W, pool=pool, budget=budget, n_cal=n_cal, cap=budget + 2)
    orc = oracle.compress(Q, K, V, window=W, pool=pool, budget=budget, n_cal=n_cal, cap=budget + 2)
    np.testing.assert_allclose(g.pooled, orc.pooled, rtol=2e-5, atol=1e-9)
    ref, _ = compare_compress(g, Q, K, V, window=W, pool=pool, budget=budget, n_cal=n_cal, orc=orc)
    q, kn, vn = wl.gen_decode_inputs(cfg, Q, steps=2)
    decode_steps_compare(g, ref, q, kn, vn, steps=2)


@pytest.mark.parametrize("calib_size", [1, 40, 300, 10 ** 6, -1])
def test_calibration_size(cuda_lib, calib_size):
    """Section 4.4's calibration size m: only the m evicted rows of highest pooled vote are calibrated
    (and offloaded); m >= the number evicted is Algorithm 1 as printed, -1 switches the calibration off."""
    from paper_2507_19906_b200 import binding as cd
    B, Hq, Hkv, L, W, pool, budget, n_cal = 2, 8, 2, 1500, 16, 7, 200, 16
    cfg = wl.small_config(B=B, Hq=Hq, Hkv=Hkv, L=L, window=W, pool=pool, budget=budget, steps=3, n_sink=2, n_heavy=40)
    Q, K, V = _inputs(cfg)
    m = None if calib_size == 10 ** 6 else max(calib_size, 0)
    orc = oracle.compress(Q, K, V, window=W, pool=pool, budget=budget, n_cal=n_cal, cap=budget + 3, calib_size=m)
    p = cd.make_params(B=B, Hq=Hq, Hkv=Hkv, L=L, window=W, pool=pool, budget=budget, n_cal=n_cal, cap=budget + 3,
                       calib_size=calib_size)
    st = cd.alloc_layer_state(p)
    dQ, dK, dV = to_dev(Q), to_dev(K), to_dev(V)
    cd.calidrop_compress(p, dQ, dK, dV, None, st.kept_idx, st.K_kept, st.V_kept, st.O_c, st.LSE_c, st.C_q,
                         st.ws_compress)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(st.kept_idx.cpu().numpy(), orc.kept_idx)      # no near-tie in this input
    np.testing.assert_array_equal(to_bits(st.C_q), orc.C_q)
    assert_close_lse(st.LSE_c.cpu().numpy(), orc.LSE_c, "LSE_c")
    assert_close_out(st.O_c.cpu().numpy(), orc.O_c, "O_c")
    if calib_size == -1:
        assert np.all(np.isneginf(st.LSE_c.cpu().numpy()))
        return
    # the calibrated rows, compacted for offloading: the same list and bit copies of the rows
    n_e = min(calib_size, L - budget)
    ev_idx = torch.empty((B, Hkv, n_e), dtype=torch.int32, device="cuda")
    K_e = torch.empty((B, Hkv, n_e, 128), dtype=torch.bfloat16, device="cuda")
    V_e = torch.empty_like(K_e)
    cd.calidrop_gather_evicted(p, dK, dV, st.kept_idx, ev_idx, K_e, V_e, st.ws_compress)
    torch.cuda.synchronize()
    want = orc.calib_idx if m is not None else np.stack(
        [[np.setdiff1d(np.arange(L - W), orc.kept_idx[b, h]) for h in range(Hkv)] for b in range(B)])
    np.testing.assert_array_equal(ev_idx.cpu().numpy(), want)
    for b in range(B):
        for h in range(Hkv):
            np.testing.assert_array_equal(to_bits(K_e)[b, h], K[b, h][want[b, h]])
            np.testing.assert_array_equal(to_bits(V_e)[b, h], V[b, h][want[b, h]])
    # and decode goes on as usual with the smaller calibration term
    g = type("R", (), {})()
    g.p, g.st, g.n_kept = p, st, budget
    ref = orc
    q, kn, vn = wl.gen_decode_inputs(cfg, Q, steps=3)
    decode_steps_compare(g, ref, q, kn, vn, steps=3)


def test_supplied_row_lse_matches_self_computed(cuda_lib):
    cfg = wl.small_config(B=1, Hq=4, Hkv=2, L=400, window=16, pool=7, budget=64)
    Q, K, V = _inputs(cfg)
    orc = oracle.compress(Q, K, V, window=16, pool=7, budget=64, n_cal=4)
    g = gpu_compress(Q, K, V, window=16, pool=7, budget=64, n_cal=4, lse_obs=orc.row_lse)
    compare_compress(g, Q, K, V, window=16, pool=7, budget=64, n_cal=4, orc=orc)


def test_budget_at_least_prefix_is_full_attention(cuda_lib):
    """Nothing evicted: LSE_c = -inf, O_c = 0, decode equals brute-force attention."""
    cfg = wl.small_config(B=1, Hq=4, Hkv=2, L=200, window=8, pool=5, budget=256)
    Q, K, V = _inputs(cfg)
    g = gpu_compress(Q, K, V, window=8, pool=5, budget=256, n_cal=2, cap=204)
    assert g.n_kept == 200
    np.testing.assert_array_equal(g.kept_idx, np.broadcast_to(np.arange(200), (1, 2, 200)))
    assert np.all(np.isneginf(g.LSE_c)) and np.all(g.O_c == 0)
    ref = oracle.compress(Q, K, V, window=8, pool=5, budget=256, n_cal=2, cap=204)
    q, kn, vn = wl.gen_decode_inputs(cfg, Q, steps=3)
    st = decode_steps_compare(g, ref, q, kn, vn, theta2=-1.0)
    assert st["applied"] == 0
    # and the GPU output against brute-force attention over the whole prompt plus the appended rows
    from paper_2507_19906_b200 import binding as cd
    out = torch.empty((1, 4, 128), dtype=torch.bfloat16, device="cuda")
    lse = torch.empty((1, 4), dtype=torch.float32, device="cuda")
    flags = torch.empty((1, 4), dtype=torch.uint8, device="cuda")
    # (the three steps above appended their rows to the GPU cache; repeat the last query without appending)
    cd.calidrop_decode(g.p, to_dev(q[2]), None, None, g.st.K_kept, g.st.V_kept, 203, g.st.O_c, g.st.LSE_c,
                       g.st.C_q, out, lse, flags, g.st.ws_decode)
    torch.cuda.synchronize()
    got = wl.bf16_bits_to_f64(to_bits(out))
    for hq in range(4):
        h = hq // 2
        Kf = np.concatenate([K[0, h], kn[:3, 0, h]])
        Vf = np.concatenate([V[0, h], vn[:3, 0, h]])
        o, l = oracle.full_attention(q[2, 0, hq][None], Kf, Vf)
        assert_close_out(got[0, hq], o[0], "nothing evicted: output vs brute-force full attention")
        assert abs(float(lse[0, hq]) - l[0]) < 1e-3


def test_query_equal_to_calibration_query_recovers_full_attention(cuda_lib):
    """Eq. 1's exact case on the GPU: q == C_q[c] => output == attention over the whole prompt."""
    cfg = wl.small_config(B=1, Hq=4, Hkv=2, L=600, window=16, pool=7, budget=80)
    Q, K, V = _inputs(cfg)
    n_cal = 4
    g = gpu_compress(Q, K, V, window=16, pool=7, budget=80, n_cal=n_cal)
    from paper_2507_19906_b200 import binding as cd
    out = torch.empty((1, 4, 128), dtype=torch.bfloat16, device="cuda")
    lse = torch.empty((1, 4), dtype=torch.float32, device="cuda")
    flags = torch.empty((1, 4), dtype=torch.uint8, device="cuda")
    for c in range(n_cal):
        qc = np.ascontiguousarray(Q[:, :, 16 - n_cal + c])
        cd.calidrop_decode(g.p, to_dev(qc), None, None, g.st.K_kept, g.st.V_kept, 80, g.st.O_c, g.st.LSE_c,
                           g.st.C_q, out, lse, flags, g.st.ws_decode)
        torch.cuda.synchronize()
        got = wl.bf16_bits_to_f64(to_bits(out))
        f = flags.cpu().numpy()
        assert np.all(f & 1 == 1) and np.all(f >> 2 == c)
        for hq in range(4):
            o, l = oracle.full_attention(qc[0, hq][None], K[0, hq // 2], V[0, hq // 2])
            assert_close_out(got[0, hq], o[0], "merged output vs brute-force full attention")
            assert abs(float(lse[0, hq]) - l[0]) < 1e-3


def test_gate_thresholds(cuda_lib):
    cfg = wl.small_config(B=2, Hq=4, Hkv=2, L=300, window=8, pool=5, budget=40)
    Q, K, V = _inputs(cfg)
    g = gpu_compress(Q, K, V, window=8, pool=5, budget=40, n_cal=8, cap=48)
    ref, _ = compare_compress(g, Q, K, V, window=8, pool=5, budget=40, n_cal=8)
    q, kn, vn = wl.gen_decode_inputs(cfg, Q, steps=2)
    never = decode_steps_compare(g, ref, q, kn, vn, theta1=0.0, theta2=1.0, steps=1, append=False)
    always = decode_steps_compare(g, ref, q, kn, vn, theta1=0.0, theta2=-1.0, steps=1, append=False)
    assert never["applied"] == 0 and always["applied"] == always["total"]
    paper = decode_steps_compare(g, ref, q, kn, vn, theta1=0.7, theta2=0.85, steps=2, append=True)
    assert paper["total"] == 2 * 2 * 4


def test_zero_query_and_determinism(cuda_lib):
    cfg = wl.small_config(B=1, Hq=4, Hkv=2, L=300, window=8, pool=5, budget=40)
    Q, K, V = _inputs(cfg)
    a = gpu_compress(Q, K, V, window=8, pool=5, budget=40, n_cal=8, cap=44)
    b = gpu_compress(Q, K, V, window=8, pool=5, budget=40, n_cal=8, cap=44)
    for name in ("kept_idx", "K_kept", "V_kept", "O_c", "LSE_c", "C_q", "vote", "pooled"):
        np.testing.assert_array_equal(getattr(a, name), getattr(b, name), err_msg=name)
    ref, _ = compare_compress(a, Q, K, V, window=8, pool=5, budget=40, n_cal=8)
    z = np.zeros((1, 1, 4, 128), dtype=np.uint16)
    st = decode_steps_compare(a, ref, z, z[:, :, :2], z[:, :, :2], steps=1, append=False)
    assert st["applied"] == 0


def test_invalid_arguments_have_no_effect(cuda_lib):
    cd = cuda_lib
    cfg = wl.small_config()
    Q, K, V = _inputs(cfg)
    good = dict(B=1, Hq=4, Hkv=2, L=300, window=8, pool=5, budget=40, n_cal=1, cap=40)
    st = cd.alloc_layer_state(cd.make_params(**good))
    dQ, dK, dV = to_dev(Q), to_dev(K), to_dev(V)
    st.kept_idx.fill_(-7)

    def call(**kw):
        p = cd.make_params(**{**good, **kw})
        return cd.calidrop_compress(p, dQ, dK, dV, None, st.kept_idx, st.K_kept, st.V_kept, st.O_c, st.LSE_c,
                                    st.C_q, st.ws_compress, check=False)

    assert call(budget=8) == cd.INVALID_ARG          # budget <= window < L
    assert call(pool=4) == cd.INVALID_ARG
    assert call(n_cal=9) == cd.INVALID_ARG
    assert call(cap=10) == cd.INVALID_ARG
    assert call(D=64) == cd.UNSUPPORTED
    assert call(Hq=18, Hkv=2) == cd.UNSUPPORTED      # G = 9
    assert call(Hq=5) == cd.INVALID_ARG
    p = cd.make_params(**good)
    assert cd.calidrop_compress(p, None, dK, dV, None, st.kept_idx, st.K_kept, st.V_kept, st.O_c, st.LSE_c,
                                st.C_q, st.ws_compress, check=False) == cd.INVALID_ARG
    assert cd.calidrop_compress(p, dQ.view(torch.uint8)[2:].view(torch.bfloat16), dK, dV, None, st.kept_idx,
                                st.K_kept, st.V_kept, st.O_c, st.LSE_c, st.C_q, st.ws_compress,
                                check=False) == cd.INVALID_ARG
    assert cd.calidrop_compress(p, dQ, dK, dV, None, st.kept_idx, st.K_kept, st.V_kept, st.O_c, st.LSE_c,
                                st.C_q, st.ws_compress[:256], check=False) == cd.WORKSPACE_TOO_SMALL
    torch.cuda.synchronize()
    assert torch.all(st.kept_idx == -7)              # failed calls launched nothing
    out = torch.empty((1, 4, 128), dtype=torch.bfloat16, device="cuda")
    dq = to_dev(np.zeros((1, 4, 128), np.uint16))
    assert cd.calidrop_decode(p, dq, None, None, st.K_kept, st.V_kept, 0, st.O_c, st.LSE_c, st.C_q, out, None,
                              None, st.ws_decode, check=False) == cd.INVALID_ARG     # empty cache
    assert cd.calidrop_decode(p, dq, None, None, st.K_kept, st.V_kept, 41, st.O_c, st.LSE_c, st.C_q, out, None,
                              None, st.ws_decode, check=False) == cd.INVALID_ARG     # beyond cap
    assert "invalid" in cd.status_string(cd.INVALID_ARG)


def test_batched_layers_match_single_layer_calls(cuda_lib):
    cd = cuda_lib
    cfg = wl.small_config(B=2, Hq=4, Hkv=2, L=260, window=8, pool=5, budget=40, layers=3)
    layers, singles = [], []
    out_b = []
    for layer in range(3):
        Q, K, V = _inputs(cfg, layer)
        g = gpu_compress(Q, K, V, window=8, pool=5, budget=40, n_cal=4, cap=42)
        q, kn, vn = wl.gen_decode_inputs(cfg, Q, layer, steps=1)
        dq, dk, dv = to_dev(q[0]), to_dev(kn[0]), to_dev(vn[0])
        Kb, Vb = g.st.K_kept.clone(), g.st.V_kept.clone()
        ob = torch.empty((2, 4, 128), dtype=torch.bfloat16, device="cuda")
        lb = torch.empty((2, 4), dtype=torch.float32, device="cuda")
        fb = torch.empty((2, 4), dtype=torch.uint8, device="cuda")
        layers.append(dict(q=dq, k_new=dk, v_new=dv, K_kept=Kb, V_kept=Vb, O_c=g.st.O_c, LSE_c=g.st.LSE_c,
                           C_q=g.st.C_q, out=ob, lse_out=lb, flags=fb))
        out_b.append((ob, lb, fb, Kb, Vb))
        os_ = torch.empty_like(ob); ls = torch.empty_like(lb); fs = torch.empty_like(fb)
        cd.calidrop_decode(g.p, dq, dk, dv, g.st.K_kept, g.st.V_kept, 40, g.st.O_c, g.st.LSE_c, g.st.C_q, os_, ls,
                           fs, g.st.ws_decode)
        singles.append((os_, ls, fs, g.st.K_kept, g.st.V_kept))
        p = g.p
    ws = torch.zeros((cd.calidrop_decode_workspace_bytes(p, 42) * 3,), dtype=torch.uint8, device="cuda")
    cd.calidrop_decode_batched(p, cd.make_decode_layers(layers), 40, ws)
    torch.cuda.synchronize()
    for (ob, lb, fb, Kb, Vb), (os_, ls, fs, Ks, Vs) in zip(out_b, singles):
        # the split factor differs between the two launches, so outputs agree to rounding only
        assert torch.allclose(ob.float(), os_.float(), atol=2e-2)
        assert torch.allclose(lb, ls, atol=1e-4)
        assert torch.equal(fb, fs)
        assert torch.equal(Kb, Ks) and torch.equal(Vb, Vs)


# ---------------------------------------------------------------- the benchmark configurations
def _run_config_full(cfg, n_cal, steps):
    Q, K, V = _inputs(cfg)
    g = gpu_compress(Q, K, V, window=cfg.window, pool=cfg.pool, budget=cfg.budget, n_cal=n_cal,
                     cap=cfg.budget + steps)
    ref, swaps = compare_compress(g, Q, K, V, window=cfg.window, pool=cfg.pool, budget=cfg.budget, n_cal=n_cal)
    q, kn, vn = wl.gen_decode_inputs(cfg, Q, steps=steps)
    st = decode_steps_compare(g, ref, q, kn, vn, steps=steps)
    return swaps, st


@pytest.mark.parametrize("n_cal", [1, 32])
def test_config1_full(cuda_lib, n_cal):
    cfg = wl.CONFIGS[1]
    swaps, st = _run_config_full(cfg, n_cal, cfg.steps)
    assert st["applied"] > 0.5 * st["total"]      # cos-sim ~0.9 > theta2: calibration is exercised


@pytest.mark.parametrize("n_cal", [1, 32])
def test_config2_full(cuda_lib, n_cal):
    cfg = wl.CONFIGS[2]
    swaps, st = _run_config_full(cfg, n_cal, cfg.steps)
    assert st["applied"] > 0.5 * st["total"]


def _sampled_units_check(cfg, layer, n_cal, units, steps, step_ids, compress_units=None):
    """Full-size GPU run through the C-ABI.  The oracle evaluates compress-and-calibrate on
    `compress_units` (default: `units`) and the decode steps `step_ids` on `units`; the sampled units
    go to the oracle as one batch, so that its loop over units runs on all host cores.
    Returns (number of heads that applied the calibration, number that did not) over the checked steps."""
    Q, K, V = _inputs(cfg, layer)
    T = steps
    g = gpu_compress(Q, K, V, window=cfg.window, pool=cfg.pool, budget=cfg.budget, n_cal=n_cal,
                     cap=cfg.budget + T)
    G = cfg.G
    q, kn, vn = wl.gen_decode_inputs(cfg, Q, layer, steps=T)
    # GPU decode over all steps, recording the sampled steps' outputs
    from paper_2507_19906_b200 import binding as cd
    p, st = g.p, g.st
    out = torch.empty((p.B, p.Hq, p.D), dtype=torch.bfloat16, device="cuda")
    lse = torch.empty((p.B, p.Hq), dtype=torch.float32, device="cuda")
    flags = torch.empty((p.B, p.Hq), dtype=torch.uint8, device="cuda")
    rec = {}
    for t in range(T):
        cd.calidrop_decode(p, to_dev(q[t]), to_dev(kn[t]), to_dev(vn[t]), st.K_kept, st.V_kept, cfg.budget + t,
                           st.O_c, st.LSE_c, st.C_q, out, lse, flags, st.ws_decode)
        if t in step_ids:
            torch.cuda.synchronize()
            rec[t] = (wl.bf16_bits_to_f64(to_bits(out)), lse.cpu().numpy(), flags.cpu().numpy())
    torch.cuda.synchronize()
    off = cd.calidrop_decode_workspace_status_offset(p)
    assert int(st.ws_decode[off:off + 4].view(torch.int32).item()) == 0, "a wait of the decode kernel ran out"

    # the sampled units as a batch of single-kv-head problems: [n, G, W, D] queries, [n, 1, L, D] keys/values
    cu = list(compress_units if compress_units is not None else units)
    assert set(units) <= set(cu)
    hsl = lambda h: slice(h * G, (h + 1) * G)
    Qs = np.ascontiguousarray(np.stack([Q[b, hsl(h)] for b, h in cu]))
    Ks = np.ascontiguousarray(np.stack([K[b, h:h + 1] for b, h in cu]))
    Vs = np.ascontiguousarray(np.stack([V[b, h:h + 1] for b, h in cu]))
    sub = type("R", (), {})()
    sub.kept_idx = np.stack([g.kept_idx[b, h:h + 1] for b, h in cu])
    sub.K_kept = np.stack([g.K_kept[b, h:h + 1] for b, h in cu])
    sub.V_kept = np.stack([g.V_kept[b, h:h + 1] for b, h in cu])
    sub.O_c = np.stack([g.O_c[b, hsl(h)] for b, h in cu])
    sub.LSE_c = np.stack([g.LSE_c[b, hsl(h)] for b, h in cu])
    sub.C_q = np.stack([g.C_q[b, hsl(h)] for b, h in cu])
    sub.n_kept, sub.cap = g.n_kept, g.cap
    ref, swaps = compare_compress(sub, Qs, Ks, Vs, window=cfg.window, pool=cfg.pool, budget=cfg.budget, n_cal=n_cal)

    applied = not_applied = 0
    for (b, h) in units:
        i = cu.index((b, h))
        hs = hsl(h)
        Kk, Vk = ref.K_kept[i:i + 1].copy(), ref.V_kept[i:i + 1].copy()
        Oc, Lc, Cq = ref.O_c[i:i + 1], ref.LSE_c[i:i + 1], ref.C_q[i:i + 1]
        for t in range(T):
            qs = np.ascontiguousarray(q[t, b:b + 1, hs])
            kns = np.ascontiguousarray(kn[t, b:b + 1, h:h + 1])
            vns = np.ascontiguousarray(vn[t, b:b + 1, h:h + 1])
            if t not in step_ids:
                Kk[0, 0, cfg.budget + t], Vk[0, 0, cfg.budget + t] = kns[0, 0], vns[0, 0]
                continue
            o = oracle.decode(qs, kns, vns, Kk, Vk, cfg.budget + t, Oc, Lc, Cq)
            gout, glse, gfl = rec[t]
            gf = gfl[b, hs]
            if not np.array_equal(gf, o.flags[0]):
                fc = (gf >> 2).astype(np.int32)[None]
                fa = (gf & 1).astype(np.int32)[None]
                for k in np.nonzero(gf != o.flags[0])[0]:
                    rho = o.rho[0, k]
                    assert abs(rho[gf[k] >> 2] - rho.max()) < 1e-4
                    assert (gf[k] & 1) == (o.flags[0, k] & 1) or abs(rho.max() - 0.85) < 1e-3
                o = oracle.decode(qs, None, None, Kk, Vk, cfg.budget + t + 1, Oc, Lc, Cq,
                                  force_c=fc, force_apply=fa)
            assert_close_out(gout[b, hs], o.out[0], f"layer {layer} unit ({b},{h}) step {t}")
            assert_close_lse(glse[b, hs], o.lse[0], f"layer {layer} unit ({b},{h}) step {t} lse")
            applied += int((gf & 1).sum())
            not_applied += int((1 - (gf & 1)).sum())
    return applied, not_applied


# ---------------------------------------------------------------- the configurations at full size
def test_config3_every_unit_and_every_decode_step(cuda_lib):
    """Config 3 as benchmarked (n_cal = W = 64): compress-and-calibrate of all 32 units against the
    oracle, and all 128 decode steps on four units (one per batch element)."""
    cfg = wl.CONFIGS[3]
    every = [(b, h) for b in range(cfg.B) for h in range(cfg.Hkv)]
    applied, _ = _sampled_units_check(cfg, 0, n_cal=64, units=[(0, 0), (1, 3), (2, 6), (3, 7)], steps=cfg.steps,
                                      step_ids=set(range(cfg.steps)), compress_units=every)
    assert applied > 0


def test_config4_every_layer(cuda_lib):
    """Config 4: each of the 32 layers at full size on the GPU, two units per layer against the oracle
    (the units move with the layer so that every batch element and kv head is visited)."""
    cfg = wl.CONFIGS[4]
    for layer in range(cfg.layers):
        units = [(layer % cfg.B, (layer // 4) % cfg.Hkv), ((layer + 3) % cfg.B, (layer + 5) % cfg.Hkv)]
        _sampled_units_check(cfg, layer, n_cal=32, units=units, steps=4, step_ids={0, 3})


def test_config5_every_unit_and_the_drift_across_the_gate(cuda_lib):
    """Config 5: all four units of the 131072-token prompt, and decode steps spread over the whole run
    of 512: the query noise grows with the step, so early steps apply the calibration and late steps,
    past the point where the similarity falls below theta2, do not.  Both must occur."""
    cfg = wl.CONFIGS[5]
    every = [(0, h) for h in range(cfg.Hkv)]
    applied, not_applied = _sampled_units_check(cfg, 0, n_cal=64, units=every, steps=cfg.steps,
                                                step_ids={0, 100, 200, 300, 400, 480, 511})
    assert applied > 0 and not_applied > 0


def test_config3_sampled_units(cuda_lib):
    cfg = wl.CONFIGS[3]
    _sampled_units_check(cfg, 0, n_cal=64, units=[(0, 0), (3, 5)], steps=8, step_ids={0, 7})


def test_config3_sampled_units_last_query_only(cuda_lib):
    cfg = wl.CONFIGS[3]
    _sampled_units_check(cfg, 0, n_cal=1, units=[(1, 7)], steps=2, step_ids={1})


def test_config5_last_query_only(cuda_lib):
    cfg = wl.CONFIGS[5]
    _sampled_units_check(cfg, 0, n_cal=1, units=[(0, 2)], steps=4, step_ids={3})


# ---------------------------------------------------------------- decode on hand-built states
@pytest.mark.parametrize("B,Hq,Hkv,kv0,steps,n_cal", [
    (1, 4, 2, 0, 6, 3),       # the cache starts empty: the first step attends to its own row alone
    (2, 8, 2, 60, 8, 2),      # the appended row crosses the first 64-row slot boundary
    (1, 7, 1, 1020, 10, 5),   # ... and a 16-row block boundary deep in a slice
    (3, 8, 8, 250, 4, 1),     # 24 units: clusters of 4, slices of about 64 rows
    (1, 4, 1, 16500, 3, 2),   # one unit, 16500 rows: two clusters per unit meet through the workspace
    (1, 8, 2, 40000, 2, 1),   # two units, 40000 rows each: four clusters per unit
])
def test_decode_ignores_cache_rows_beyond_kv_len(cuda_lib, B, Hq, Hkv, kv0, steps, n_cal):
    """The cache rows at and beyond kv_len belong to the caller and may hold anything; here they
    hold NaN bit patterns.  Every step must still match the oracle, which never reads them."""
    from paper_2507_19906_b200 import binding as cd
    rng = np.random.Generator(np.random.Philox(key=[77, B * 1000 + kv0]))
    D, cap = 128, max(kv0 + steps, 64)
    bits = lambda x: wl.f32_to_bf16_bits(np.ascontiguousarray(x, dtype=np.float32))
    budget = min(cap, max(kv0, 16))
    p = cd.make_params(B=B, Hq=Hq, Hkv=Hkv, L=budget + 64, window=8, pool=7, budget=budget, n_cal=n_cal, cap=cap)
    st = cd.alloc_layer_state(p)
    Kk = np.full((B, Hkv, cap, D), 0x7FC0, dtype=np.uint16)   # quiet NaN everywhere ...
    Vk = np.full((B, Hkv, cap, D), 0x7FC0, dtype=np.uint16)
    Kk[:, :, :kv0] = bits(rng.standard_normal((B, Hkv, kv0, D)))   # ... except the valid rows
    Vk[:, :, :kv0] = bits(rng.standard_normal((B, Hkv, kv0, D)))
    Cq = bits(rng.standard_normal((B, Hq, n_cal, D)))
    Oc = rng.standard_normal((B, Hq, n_cal, D)).astype(np.float32)
    Lc = (rng.standard_normal((B, Hq, n_cal)) + 3.0).astype(np.float32)
    st.K_kept.copy_(to_dev(Kk)); st.V_kept.copy_(to_dev(Vk)); st.C_q.copy_(to_dev(Cq))
    st.O_c.copy_(torch.from_numpy(Oc)); st.LSE_c.copy_(torch.from_numpy(Lc))
    out = torch.empty((B, Hq, D), dtype=torch.bfloat16, device="cuda")
    lse = torch.empty((B, Hq), dtype=torch.float32, device="cuda")
    flags = torch.empty((B, Hq), dtype=torch.uint8, device="cuda")
    p.theta1, p.theta2 = 0.7, -1.0                                  # always merge: O_c and LSE_c matter
    for t in range(steps):
        # queries close to a calibration query half of the time, so that both rows get chosen
        q = bits(wl.bf16_bits_to_f32(Cq[:, :, t % n_cal]) + 0.5 * rng.standard_normal((B, Hq, D)).astype(np.float32))
        kn, vn = bits(rng.standard_normal((B, Hkv, D))), bits(rng.standard_normal((B, Hkv, D)))
        cd.calidrop_decode(p, to_dev(q), to_dev(kn), to_dev(vn), st.K_kept, st.V_kept, kv0 + t, st.O_c, st.LSE_c,
                           st.C_q, out, lse, flags, st.ws_decode)
        torch.cuda.synchronize()
        o = oracle.decode(q, kn, vn, Kk, Vk, kv0 + t, Oc, Lc, Cq, theta1=0.7, theta2=-1.0)
        got = wl.bf16_bits_to_f64(to_bits(out))
        gf = flags.cpu().numpy()
        if not np.array_equal(gf >> 2, o.flags >> 2):
            # the chosen calibration row may differ only when the two similarities are within 1e-4;
            # the oracle is then re-evaluated under the GPU's choice
            force_c = np.full((B, Hq), -1, dtype=np.int32)
            for b, hq in zip(*np.nonzero((gf >> 2) != (o.flags >> 2))):
                gc, oc = int(gf[b, hq] >> 2), int(o.flags[b, hq] >> 2)
                assert abs(o.rho[b, hq, gc] - o.rho[b, hq, oc]) < 1e-4, "calibration row differs beyond a near-tie"
                force_c[b, hq] = gc
            o = oracle.decode(q, None, None, Kk, Vk, kv0 + t + 1, Oc, Lc, Cq, theta1=0.7, theta2=-1.0,
                              force_c=force_c)
        assert_close_out(got, o.out, f"step {t}")
        assert_close_lse(lse.cpu().numpy(), o.lse, f"step {t} lse")
        # the appended row reached the cache, bit for bit, and nothing else was written
        np.testing.assert_array_equal(to_bits(st.K_kept)[:, :, :kv0 + t + 1], Kk[:, :, :kv0 + t + 1])
        np.testing.assert_array_equal(to_bits(st.V_kept)[:, :, :kv0 + t + 1], Vk[:, :, :kv0 + t + 1])
        np.testing.assert_array_equal(to_bits(st.K_kept)[:, :, kv0 + t + 1:], Kk[:, :, kv0 + t + 1:])


def test_batched_layers_with_several_clusters_per_unit(cuda_lib):
    """Two layers of one unit with 17000 cached rows in one launch: every (layer, unit) is split over
    two clusters that meet through the workspace, each layer with its own counters and partials.
    Checked against the oracle, twice on the same workspace (the counters must come back to zero)."""
    cd = cuda_lib
    rng = np.random.Generator(np.random.Philox(key=[91, 5]))
    B, Hq, Hkv, D, kv0, n_cal, NL = 1, 4, 1, 128, 17000, 2, 2
    cap = kv0 + 2
    bits = lambda x: wl.f32_to_bf16_bits(np.ascontiguousarray(x, dtype=np.float32))
    p = cd.make_params(B=B, Hq=Hq, Hkv=Hkv, L=kv0 + 64, window=8, pool=7, budget=kv0, n_cal=n_cal, cap=cap)
    p.theta1, p.theta2 = 0.7, -1.0
    ws = torch.zeros((cd.calidrop_decode_workspace_bytes(p, cap) * NL,), dtype=torch.uint8, device="cuda")
    host, layers = [], []
    for _ in range(NL):
        Kk = np.zeros((B, Hkv, cap, D), dtype=np.uint16); Vk = np.zeros_like(Kk)
        Kk[:, :, :kv0] = bits(rng.standard_normal((B, Hkv, kv0, D)))
        Vk[:, :, :kv0] = bits(rng.standard_normal((B, Hkv, kv0, D)))
        Cq = bits(rng.standard_normal((B, Hq, n_cal, D)))
        Oc = rng.standard_normal((B, Hq, n_cal, D)).astype(np.float32)
        Lc = (rng.standard_normal((B, Hq, n_cal)) + 9.0).astype(np.float32)
        dev = dict(K_kept=to_dev(Kk), V_kept=to_dev(Vk), C_q=to_dev(Cq), O_c=torch.from_numpy(Oc).cuda(),
                   LSE_c=torch.from_numpy(Lc).cuda(),
                   out=torch.empty((B, Hq, D), dtype=torch.bfloat16, device="cuda"),
                   lse_out=torch.empty((B, Hq), dtype=torch.float32, device="cuda"),
                   flags=torch.empty((B, Hq), dtype=torch.uint8, device="cuda"))
        host.append((Kk, Vk, Cq, Oc, Lc)); layers.append(dev)
    for t in range(2):
        step = []
        for dev, (Kk, Vk, Cq, Oc, Lc) in zip(layers, host):
            q = bits(wl.bf16_bits_to_f32(Cq[:, :, t % n_cal]) + 0.5 * rng.standard_normal((B, Hq, D)).astype(np.float32))
            kn, vn = bits(rng.standard_normal((B, Hkv, D))), bits(rng.standard_normal((B, Hkv, D)))
            dev.update(q=to_dev(q), k_new=to_dev(kn), v_new=to_dev(vn))
            step.append((q, kn, vn))
        cd.calidrop_decode_batched(p, cd.make_decode_layers(layers), kv0 + t, ws)
        torch.cuda.synchronize()
        off = cd.calidrop_decode_workspace_status_offset(p)
        assert int(ws[off:off + 4].view(torch.int32).item()) == 0
        for dev, (Kk, Vk, Cq, Oc, Lc), (q, kn, vn) in zip(layers, host, step):
            o = oracle.decode(q, kn, vn, Kk, Vk, kv0 + t, Oc, Lc, Cq, theta1=0.7, theta2=-1.0)
            same = (dev["flags"].cpu().numpy() >> 2) == (o.flags >> 2)
            assert same.all()
            assert_close_out(wl.bf16_bits_to_f64(to_bits(dev["out"])), o.out, f"step {t}")
            assert_close_lse(dev["lse_out"].cpu().numpy(), o.lse, f"step {t} lse")
            np.testing.assert_array_equal(to_bits(dev["K_kept"]), Kk)


# ---------------------------------------------------------------- a kept list chosen by the caller
def _streaming_indices(B, Hkv, L, budget, n_sink):
    """Index rule of a sink-plus-recent cache: the first n_sink rows and the most recent ones."""
    idx = np.concatenate([np.arange(n_sink), np.arange(L - (budget - n_sink), L)]).astype(np.int32)
    return np.broadcast_to(idx, (B, Hkv, budget)).copy()


@pytest.mark.parametrize("B,Hq,Hkv,L,W,budget,n_cal,rule,supply_lse", [
    (1, 4, 2, 700, 16, 96, 4, "streaming", False),
    (2, 8, 2, 1500, 32, 256, 32, "random", False),     # two 128-row calibration blocks per kv head
    (1, 7, 1, 3000, 64, 400, 64, "streaming", True),   # G = 7, row LSE supplied by the caller
])
def test_calibrate_with_a_supplied_kept_list(cuda_lib, B, Hq, Hkv, L, W, budget, n_cal, rule, supply_lse):
    cd = cuda_lib
    cfg = wl.small_config(B=B, Hq=Hq, Hkv=Hkv, L=L, window=W, pool=7, budget=budget, steps=3,
                          n_sink=4, n_heavy=max(1, L // 50))
    Q, K, V = _inputs(cfg)
    if rule == "streaming":
        kept = _streaming_indices(B, Hkv, L, budget, 32)
    else:
        rng = np.random.Generator(np.random.Philox(key=[5, L]))
        kept = np.stack([np.stack([np.sort(np.concatenate([
            rng.choice(L - W, size=budget - W, replace=False), np.arange(L - W, L)])).astype(np.int32)
            for _ in range(Hkv)]) for _ in range(B)])
    T = 3
    p = cd.make_params(B=B, Hq=Hq, Hkv=Hkv, L=L, window=W, pool=7, budget=budget, n_cal=n_cal, cap=budget + T)
    st = cd.alloc_layer_state(p)
    ref = oracle.calibrate_given_indices(Q, K, V, kept, n_cal=n_cal, cap=budget + T)
    lse = None
    if supply_lse:
        lse = torch.from_numpy(oracle.compress(Q, K, V, window=W, pool=7, budget=budget, n_cal=n_cal)
                               .row_lse.astype(np.float32)).cuda()
    cd.calidrop_calibrate(p, to_dev(Q), to_dev(K), to_dev(V), lse, torch.from_numpy(kept).cuda(), st.K_kept,
                          st.V_kept, st.O_c, st.LSE_c, st.C_q, st.ws_compress)
    torch.cuda.synchronize()
    lay = cd.calidrop_compress_workspace_layout(p)
    assert int(st.ws_compress[lay.status_offset:lay.status_offset + 4].view(torch.int32).item()) == 0
    np.testing.assert_array_equal(to_bits(st.K_kept)[:, :, :budget], ref.K_kept[:, :, :budget])
    np.testing.assert_array_equal(to_bits(st.V_kept)[:, :, :budget], ref.V_kept[:, :, :budget])
    np.testing.assert_array_equal(to_bits(st.C_q), ref.C_q)
    assert_close_lse(st.LSE_c.cpu().numpy(), ref.LSE_c, "LSE_c")
    assert_close_out(st.O_c.cpu().numpy(), ref.O_c, "O_c")
    # and the decode steps that follow use this state like any other
    from types import SimpleNamespace
    g = SimpleNamespace(st=st, p=p, n_kept=budget)
    q, kn, vn = wl.gen_decode_inputs(cfg, Q, steps=T)
    res = decode_steps_compare(g, ref, q, kn, vn, steps=T)
    assert res["total"] == T * B * Hq


# ---------------------------------------------------------------- the recompute branch (Algorithm 2, lines 3-8)
@pytest.mark.parametrize("B,Hq,Hkv,L,W,budget,n_cal,slot", [
    (1, 4, 2, 600, 16, 80, 1, 0),          # the paper's single calibration query
    (2, 8, 2, 1500, 32, 256, 4, 2),        # G = 4, one of four rows rewritten
    (1, 7, 1, 20000, 64, 2048, 64, 63),    # one unit, 17952 evicted rows: two clusters per unit
])
def test_gather_evicted_and_recalibrate(cuda_lib, B, Hq, Hkv, L, W, budget, n_cal, slot):
    cd = cuda_lib
    cfg = wl.small_config(B=B, Hq=Hq, Hkv=Hkv, L=L, window=W, pool=7, budget=budget, steps=2,
                          n_sink=4, n_heavy=max(1, L // 50))
    Q, K, V = _inputs(cfg)
    g = gpu_compress(Q, K, V, window=W, pool=7, budget=budget, n_cal=n_cal, cap=budget + 2, keep_inputs=True)
    n_e = L - budget
    ev_idx = torch.empty((B, Hkv, n_e), dtype=torch.int32, device="cuda")
    K_e = torch.empty((B, Hkv, n_e, 128), dtype=torch.bfloat16, device="cuda")
    V_e = torch.empty_like(K_e)
    cd.calidrop_gather_evicted(g.p, g.dK, g.dV, g.st.kept_idx, ev_idx, K_e, V_e, g.st.ws_compress)
    torch.cuda.synchronize()
    ev = ev_idx.cpu().numpy()
    for b in range(B):
        for h in range(Hkv):
            want = np.setdiff1d(np.arange(L - W), g.kept_idx[b, h])     # ascending complement among candidates
            np.testing.assert_array_equal(ev[b, h], want)
            np.testing.assert_array_equal(to_bits(K_e)[b, h], K[b, h][want])
            np.testing.assert_array_equal(to_bits(V_e)[b, h], V[b, h][want])
    # a query far from every calibration query, as in the branch's condition
    rng = np.random.Generator(np.random.Philox(key=[11, L]))
    q = wl.f32_to_bf16_bits(rng.standard_normal((B, Hq, 128)).astype(np.float32))
    O_before, L_before, C_before = g.st.O_c.clone(), g.st.LSE_c.clone(), g.st.C_q.clone()
    cd.calidrop_recalibrate(g.p, to_dev(q), K_e, V_e, n_e, slot, g.st.O_c, g.st.LSE_c, g.st.C_q, g.st.ws_decode)
    torch.cuda.synchronize()
    off = cd.calidrop_decode_workspace_status_offset(g.p)
    assert int(g.st.ws_decode[off:off + 4].view(torch.int32).item()) == 0
    G = Hq // Hkv
    for b in range(B):
        for hq in range(Hq):
            h = hq // G
            o, l = oracle.full_attention(q[b, hq][None], K[b, h][ev[b, h]], V[b, h][ev[b, h]])
            assert_close_out(g.st.O_c[b, hq, slot].cpu().numpy(), o[0], "recomputed O_c")
            assert abs(float(g.st.LSE_c[b, hq, slot]) - l[0]) < 1e-3
    np.testing.assert_array_equal(to_bits(g.st.C_q)[:, :, slot], q)
    keep = [c for c in range(n_cal) if c != slot]                      # the other rows are untouched
    assert torch.equal(g.st.O_c[:, :, keep], O_before[:, :, keep])
    assert torch.equal(g.st.LSE_c[:, :, keep], L_before[:, :, keep])
    assert torch.equal(g.st.C_q[:, :, keep], C_before[:, :, keep])
    # the repeated decode step now finds rho = 1 with the new row and merges: the result is the
    # attention of q over the kept and the evicted rows together, i.e. over the whole prompt
    out = torch.empty((B, Hq, 128), dtype=torch.bfloat16, device="cuda")
    flags = torch.empty((B, Hq), dtype=torch.uint8, device="cuda")
    cd.calidrop_decode(g.p, to_dev(q), None, None, g.st.K_kept, g.st.V_kept, budget, g.st.O_c, g.st.LSE_c, g.st.C_q,
                       out, None, flags, g.st.ws_decode)
    torch.cuda.synchronize()
    f = flags.cpu().numpy()
    assert np.all(f & 1 == 1) and np.all(f & 2 == 0)
    got = wl.bf16_bits_to_f64(to_bits(out))
    for b in range(B):
        for hq in range(Hq):
            o, _ = oracle.full_attention(q[b, hq][None], K[b, hq // G], V[b, hq // G])
            assert_close_out(got[b, hq], o[0], "decode after the recompute vs attention over the whole prompt")


def test_offload_and_reload_of_the_evicted_rows_beside_decode(cuda_lib):
    """Algorithm 1 line 4 / Algorithm 2 line 4: the compacted evicted rows go to page-locked host
    memory on a copy stream and come back on it, bit for bit, while decode steps run on the compute
    stream; the decode outputs are the same as without the transfer, and a recompute from the
    reloaded rows equals one from the rows that never left."""
    cd = cuda_lib
    B, Hq, Hkv, L, W, budget, n_cal = 2, 8, 2, 6000, 32, 512, 32
    cfg = wl.small_config(B=B, Hq=Hq, Hkv=Hkv, L=L, window=W, pool=7, budget=budget, steps=6, n_sink=4, n_heavy=100)
    Q, K, V = _inputs(cfg)
    T = 6
    g = gpu_compress(Q, K, V, window=W, pool=7, budget=budget, n_cal=n_cal, cap=budget + T, keep_inputs=True)
    p, st = g.p, g.st
    n_e = L - budget
    ev_idx = torch.empty((B, Hkv, n_e), dtype=torch.int32, device="cuda")
    K_e = torch.empty((B, Hkv, n_e, 128), dtype=torch.bfloat16, device="cuda")
    V_e = torch.empty_like(K_e)
    K_h = torch.empty(K_e.shape, dtype=torch.bfloat16).pin_memory()
    V_h = torch.empty(V_e.shape, dtype=torch.bfloat16).pin_memory()
    main, side = torch.cuda.current_stream(), torch.cuda.Stream()
    gathered, offloaded, reloaded = torch.cuda.Event(), torch.cuda.Event(), torch.cuda.Event()
    cd.calidrop_gather_evicted(p, g.dK, g.dV, st.kept_idx, ev_idx, K_e, V_e, st.ws_compress)
    gathered.record(main)
    offloaded.record(side); reloaded.record(side)          # (creates the handles; they are recorded again below)
    cd.calidrop_offload_evicted(p, n_e, K_e, V_e, K_h, V_h, side, wait_event=gathered, done_event=offloaded)
    offloaded.synchronize()
    K_ref, V_ref = K_e.clone(), V_e.clone()
    assert torch.equal(K_h, K_ref.cpu()) and torch.equal(V_h, V_ref.cpu())
    # decode steps without any transfer, on copies of the cache
    q, kn, vn = wl.gen_decode_inputs(cfg, Q, steps=T)
    dq, dk, dv = [to_dev(x) for x in q], [to_dev(x) for x in kn], [to_dev(x) for x in vn]

    def run_steps(Kc, Vc):
        outs = []
        for t in range(T):
            o = torch.empty((B, Hq, 128), dtype=torch.bfloat16, device="cuda")
            cd.calidrop_decode(p, dq[t], dk[t], dv[t], Kc, Vc, budget + t, st.O_c, st.LSE_c, st.C_q, o, None, None,
                               st.ws_decode)
            outs.append(o)
        return outs

    quiet = run_steps(st.K_kept.clone(), st.V_kept.clone())
    torch.cuda.synchronize()
    # the device copy is dropped (overwritten), then reloaded on the side stream while decode runs
    K_e.zero_(); V_e.zero_()
    torch.cuda.synchronize()
    cd.calidrop_reload_evicted(p, n_e, K_h, V_h, K_e, V_e, side, wait_event=None, done_event=reloaded)
    busy = run_steps(st.K_kept.clone(), st.V_kept.clone())
    main.wait_event(reloaded)                              # the compute stream may read the rows from here on
    assert torch.equal(K_e, K_ref) and torch.equal(V_e, V_ref)
    for a, b in zip(quiet, busy):
        assert torch.equal(a, b)
    off = cd.calidrop_decode_workspace_status_offset(p)
    assert int(st.ws_decode[off:off + 4].view(torch.int32).item()) == 0
    # a recompute from the reloaded rows
    rng = np.random.Generator(np.random.Philox(key=[12, L]))
    qr = wl.f32_to_bf16_bits(rng.standard_normal((B, Hq, 128)).astype(np.float32))
    cd.calidrop_recalibrate(p, to_dev(qr), K_e, V_e, n_e, 5, st.O_c, st.LSE_c, st.C_q, st.ws_decode)
    torch.cuda.synchronize()
    ev = ev_idx.cpu().numpy()
    for b in range(B):
        for hq in range(Hq):
            h = hq // (Hq // Hkv)
            o, l = oracle.full_attention(qr[b, hq][None], K[b, h][ev[b, h]], V[b, h][ev[b, h]])
            assert_close_out(st.O_c[b, hq, 5].cpu().numpy(), o[0], "O_c recomputed from the reloaded rows")
            assert abs(float(st.LSE_c[b, hq, 5]) - l[0]) < 1e-3
    # argument checks
    assert cd.calidrop_offload_evicted(p, 0, K_e, V_e, K_h, V_h, side, check=False) == cd.INVALID_ARG
    assert cd.calidrop_reload_evicted(p, n_e, None, V_h, K_e, V_e, side, check=False) == cd.INVALID_ARG


def test_streaming_and_h2o_kept_lists_from_the_library_feed_the_calibration(cuda_lib):
    """The paper applies CaliDrop on top of StreamingLLM and H2O too (Sections 4.1.2-4.1.3): their kept
    lists, written on the device by the library, equal the oracle's, and calidrop_calibrate on them
    matches the oracle's calibration over the rows those rules evict."""
    cd = cuda_lib
    B, Hq, Hkv, L, W, budget, n_cal = 2, 4, 2, 700, 16, 128, 4
    G = Hq // Hkv
    cfg = wl.small_config(B=B, Hq=Hq, Hkv=Hkv, L=L, window=W, pool=1, budget=budget, steps=2, n_sink=4, n_heavy=14)
    Q, K, V = _inputs(cfg)
    p = cd.make_params(B=B, Hq=Hq, Hkv=Hkv, L=L, window=W, pool=1, budget=budget, n_cal=n_cal, cap=budget + 2)
    st = cd.alloc_layer_state(p)
    dQ, dK, dV = to_dev(Q), to_dev(K), to_dev(V)
    # H2O's accumulated attention needs every prompt query: a seeded full-query tensor whose last W rows are Q_obs
    rng = np.random.Generator(np.random.Philox(key=[31, 7]))
    scores = np.zeros((B, Hkv, L), dtype=np.float32)
    for b in range(B):
        for h in range(Hkv):
            Qfull = wl.f32_to_bf16_bits(rng.standard_normal((G, L, 128)).astype(np.float32))
            Qfull[:, L - W:] = Q[b, h * G:(h + 1) * G]
            scores[b, h] = oracle.accumulated_attention(Qfull, K[b, h]).astype(np.float32)
    lists = {}
    cd.calidrop_select_streaming(p, 32, st.kept_idx)
    torch.cuda.synchronize()
    lists["streaming"] = st.kept_idx.cpu().numpy().copy()
    np.testing.assert_array_equal(lists["streaming"], np.broadcast_to(oracle.streaming_indices(L, budget, 32), (B, Hkv, budget)))
    cd.calidrop_select_from_scores(p, torch.from_numpy(scores).cuda(), budget // 2, st.kept_idx, st.ws_compress)
    torch.cuda.synchronize()
    lists["h2o"] = st.kept_idx.cpu().numpy().copy()
    for b in range(B):
        for h in range(Hkv):
            # fp32 scores on both sides: the order is the same bit for bit
            np.testing.assert_array_equal(lists["h2o"][b, h], oracle.select_from_scores(scores[b, h], tail=budget // 2, budget=budget))
    for name, kept in lists.items():
        st.kept_idx.copy_(torch.from_numpy(kept))
        cd.calidrop_calibrate(p, dQ, dK, dV, None, st.kept_idx, st.K_kept, st.V_kept, st.O_c, st.LSE_c, st.C_q,
                              st.ws_compress)
        torch.cuda.synchronize()
        ref = oracle.calibrate_given_indices(Q, K, V, kept, n_cal=n_cal, cap=budget + 2)
        np.testing.assert_array_equal(to_bits(st.K_kept)[:, :, :budget], ref.K_kept[:, :, :budget])
        assert_close_lse(st.LSE_c.cpu().numpy(), ref.LSE_c, f"{name}: LSE_c")
        assert_close_out(st.O_c.cpu().numpy(), ref.O_c, f"{name}: O_c")
    # argument checks
    assert cd.calidrop_select_streaming(p, budget, st.kept_idx, check=False) == cd.INVALID_ARG
    assert cd.calidrop_select_from_scores(p, torch.from_numpy(scores).cuda(), W - 1, st.kept_idx, st.ws_compress,
                                          check=False) == cd.INVALID_ARG


@pytest.mark.parametrize("B,Hq,Hkv,L", [(1, 4, 2, 333), (2, 6, 2, 700), (1, 8, 1, 1100)])
def test_h2o_accumulated_scores_from_the_library(cuda_lib, B, Hq, Hkv, L):
    """H2O's importance measure (Section 4.1.2): the column sums of the causal attention of every prompt
    query, per kv head, computed by the library from Q and K, against the oracle's definition; the kept
    list that the library then selects from ITS scores equals the oracle's list from the oracle's scores
    up to swaps of rows whose oracle scores are closer than the fp32 arithmetic resolves."""
    cd = cuda_lib
    G, W, budget = Hq // Hkv, 16, 128
    rng = np.random.Generator(np.random.Philox(key=[41, L]))
    Qf = wl.f32_to_bf16_bits(rng.standard_normal((B, Hq, L, 128)).astype(np.float32))
    Kb = wl.f32_to_bf16_bits(rng.standard_normal((B, Hkv, L, 128)).astype(np.float32))
    Kb[:, :, ::37] = wl.f32_to_bf16_bits(2.5 * wl.bf16_bits_to_f32(Kb[:, :, ::37]))   # some heavy hitters
    p = cd.make_params(B=B, Hq=Hq, Hkv=Hkv, L=L, window=W, pool=1, budget=budget, n_cal=1, cap=budget + 2)
    st = cd.alloc_layer_state(p)
    ws = torch.empty((cd.calidrop_accumulated_scores_workspace_bytes(p),), dtype=torch.uint8, device="cuda")
    scores = torch.full((B, Hkv, L), -1.0, dtype=torch.float32, device="cuda")
    runs = []
    for _ in range(2):                                  # twice: the result is reproducible bit for bit
        cd.calidrop_accumulated_scores(p, to_dev(Qf), to_dev(Kb), scores, ws)
        torch.cuda.synchronize()
        runs.append(scores.cpu().numpy().copy())
    np.testing.assert_array_equal(runs[0], runs[1])
    got = runs[0]
    ref = np.stack([np.stack([oracle.accumulated_attention(Qf[b, h * G:(h + 1) * G], Kb[b, h]) for h in range(Hkv)])
                    for b in range(B)])
    # every query's attention sums to one: the scores of a kv head sum to G * L
    np.testing.assert_allclose(ref.sum(-1), G * L, rtol=1e-9)
    np.testing.assert_allclose(got, ref, rtol=2e-5, atol=1e-6)
    np.testing.assert_allclose(got.sum(-1, dtype=np.float64), G * L, rtol=1e-5)
    cd.calidrop_select_from_scores(p, scores, budget // 2, st.kept_idx, st.ws_compress)
    torch.cuda.synchronize()
    kept = st.kept_idx.cpu().numpy()
    for b in range(B):
        for h in range(Hkv):
            want = oracle.select_from_scores(ref[b, h].astype(np.float32), tail=budget // 2, budget=budget)
            a, w = set(kept[b, h].tolist()), set(want.tolist())
            assert len(a) == budget and np.all(np.diff(kept[b, h]) > 0)
            if a != w:                                  # only near-ties of the oracle's scores may swap
                thr = min(ref[b, h][t] for t in w if t < L - budget // 2)
                for t in a ^ w:
                    assert abs(ref[b, h][t] - thr) <= 2e-5 * thr, (b, h, t, ref[b, h][t], thr)
    # argument checks
    small = torch.empty((16,), dtype=torch.uint8, device="cuda")
    assert cd.calidrop_accumulated_scores(p, to_dev(Qf), to_dev(Kb), scores, small, check=False) == cd.WORKSPACE_TOO_SMALL
    assert cd.calidrop_accumulated_scores(p, None, to_dev(Kb), scores, ws, check=False) == cd.INVALID_ARG


def test_calls_enqueued_back_to_back_give_the_results_of_calls_run_one_at_a_time(cuda_lib):
    """The kernels of a compress call start beside the end of their predecessors (programmatic dependent
    launch) and a decode launch prefetches ahead of its dependency wait: a stream of calls with no
    synchronisation between them, on one shared workspace, must leave exactly what the same calls leave
    when each is waited for."""
    cd = cuda_lib
    B, Hq, Hkv, L, W, pool, budget, n_cal = 2, 8, 2, 2300, 32, 7, 256, 32
    cfgs = [wl.small_config(B=B, Hq=Hq, Hkv=Hkv, L=L, window=W, pool=pool, budget=budget, steps=3, n_heavy=24,
                            seed=s) for s in (5, 6)]
    inputs = [tuple(to_dev(x) for x in _inputs(c)) for c in cfgs]
    T = 3
    p = cd.make_params(B=B, Hq=Hq, Hkv=Hkv, L=L, window=W, pool=pool, budget=budget, n_cal=n_cal, cap=budget + T)
    dec = [tuple(to_dev(x) for x in wl.gen_decode_inputs(c, wl.gen_q_obs(c), steps=T)) for c in cfgs]

    def run(sync):
        states = [cd.alloc_layer_state(p) for _ in range(2)]
        for st in states:
            st.ws_compress = states[0].ws_compress          # one workspace for every call
        outs = []
        for rnd in range(3):
            for i, (st, (dQ, dK, dV)) in enumerate(zip(states, inputs)):
                cd.calidrop_compress(p, dQ, dK, dV, None, st.kept_idx, st.K_kept, st.V_kept, st.O_c, st.LSE_c, st.C_q,
                                     st.ws_compress)
                if sync:
                    torch.cuda.synchronize()
                q, kn, vn = dec[i]
                for t in range(T):
                    o = torch.empty((B, Hq, 128), dtype=torch.bfloat16, device="cuda")
                    cd.calidrop_decode(p, q[t], kn[t], vn[t], st.K_kept, st.V_kept, budget + t, st.O_c, st.LSE_c,
                                       st.C_q, o, None, None, st.ws_decode)
                    if sync:
                        torch.cuda.synchronize()
                    outs.append(o)
        torch.cuda.synchronize()
        lay = cd.calidrop_compress_workspace_layout(p)
        assert int(states[0].ws_compress[lay.status_offset: lay.status_offset + 4].view(torch.int32).item()) == 0
        return states, outs

    ref_states, ref_outs = run(sync=True)
    got_states, got_outs = run(sync=False)
    for a, b in zip(ref_states, got_states):
        assert torch.equal(a.kept_idx, b.kept_idx)
        assert torch.equal(a.K_kept, b.K_kept) and torch.equal(a.V_kept, b.V_kept)
        assert torch.equal(a.O_c, b.O_c) and torch.equal(a.LSE_c, b.LSE_c) and torch.equal(a.C_q, b.C_q)
    for a, b in zip(ref_outs, got_outs):
        assert torch.equal(a, b)


# ---------------------------------------------------------------- seeded random shapes
def _random_shapes(n, seed):
    rng = np.random.Generator(np.random.Philox(key=[seed, 1]))
    out = []
    for _ in range(n):
        Hkv = int(rng.integers(1, 5))
        G = int(rng.integers(1, 9))
        B = int(rng.integers(1, 4))
        W = int(rng.choice([1, 2, 4, 8, 16, 32, 64]))
        if G * W > 512:
            W = 512 // G
        L = int(rng.integers(W + 40, 2600))
        budget = int(rng.integers(W + 1, min(L, W + 700)))
        pool = int(rng.choice([1, 3, 5, 7]))
        n_cal = int(rng.integers(1, W + 1))
        out.append((B, Hkv * G, Hkv, L, W, pool, budget, n_cal))
    return out


@pytest.mark.parametrize("B,Hq,Hkv,L,W,pool,budget,n_cal", _random_shapes(16, 2507))
def test_compress_and_decode_random_shapes(cuda_lib, B, Hq, Hkv, L, W, pool, budget, n_cal):
    cfg = wl.small_config(B=B, Hq=Hq, Hkv=Hkv, L=L, window=W, pool=pool, budget=budget, steps=3,
                          n_sink=2, n_heavy=max(1, L // 50))
    Q, K, V = _inputs(cfg)
    T = 3
    g = gpu_compress(Q, K, V, window=W, pool=pool, budget=budget, n_cal=n_cal, cap=budget + T)
    ref, _ = compare_compress(g, Q, K, V, window=W, pool=pool, budget=budget, n_cal=n_cal)
    q, kn, vn = wl.gen_decode_inputs(cfg, Q, steps=T)
    st = decode_steps_compare(g, ref, q, kn, vn, steps=T)
    assert st["total"] == T * B * Hq
