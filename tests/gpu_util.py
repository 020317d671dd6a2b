"""Helpers for the GPU parity tests: run the C-ABI path on numpy inputs, compare with the oracle."""
from __future__ import annotations

from types import SimpleNamespace

import numpy as np
import torch

import oracle
from paper_2507_19906_b200 import binding as cd
from paper_2507_19906_b200 import workload as wl

OUT_MAX_ABS, OUT_MEAN_ABS, LSE_ABS = 2e-2, 2e-3, 1e-3   # bf16 outputs and O_c: max-abs, mean-abs; log-sum-exps: abs
SWAP_REL = 1e-5                                         # allowed near-tie swaps in the kept set


def to_dev(bits: np.ndarray) -> torch.Tensor:
    """uint16 bf16 bit patterns -> CUDA bf16 tensor."""
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def to_bits(t: torch.Tensor) -> np.ndarray:
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def gpu_compress(Q_obs, K, V, *, window, pool, budget, n_cal=1, cap=None, lse_obs=None, theta1=0.7,
                 theta2=0.85, keep_inputs=False):
    B, Hq, W, D = Q_obs.shape
    _, Hkv, L, _ = K.shape
    n_kept = min(budget, L)
    cap = cap or n_kept
    p = cd.make_params(B=B, Hq=Hq, Hkv=Hkv, L=L, window=window, pool=pool, budget=budget, n_cal=n_cal,
                       cap=cap, theta1=theta1, theta2=theta2)
    st = cd.alloc_layer_state(p)
    dQ, dK, dV = to_dev(Q_obs), to_dev(K), to_dev(V)
    dl = None if lse_obs is None else torch.from_numpy(np.ascontiguousarray(lse_obs, dtype=np.float32)).cuda()
    cd.calidrop_compress(p, dQ, dK, dV, dl, st.kept_idx, st.K_kept, st.V_kept, st.O_c, st.LSE_c, st.C_q,
                         st.ws_compress)
    torch.cuda.synchronize()
    lay = cd.calidrop_compress_workspace_layout(p)
    n_cand = max(L - W, 0)

    def ws_f32(off, n):
        return st.ws_compress[off: off + 4 * n].view(torch.float32).cpu().numpy()

    status = int(st.ws_compress[lay.status_offset: lay.status_offset + 4].view(torch.int32).item())
    assert status == 0, f"a compress kernel gave up waiting on its pipeline (code {status})"

    r = SimpleNamespace(
        p=p, st=st,
        kept_idx=st.kept_idx.cpu().numpy(), K_kept=to_bits(st.K_kept), V_kept=to_bits(st.V_kept),
        O_c=st.O_c.cpu().numpy(), LSE_c=st.LSE_c.cpu().numpy(), C_q=to_bits(st.C_q),
        vote=ws_f32(lay.vote_offset, B * Hkv * n_cand).reshape(B, Hkv, n_cand) if budget < L else None,
        pooled=ws_f32(lay.pooled_offset, B * Hkv * n_cand).reshape(B, Hkv, n_cand) if budget < L else None,
        row_lse=ws_f32(lay.row_lse_offset, B * Hq * W).reshape(B, Hq, W) if budget < L else None,
        n_kept=n_kept, cap=cap,
    )
    if keep_inputs:
        r.dQ, r.dK, r.dV = dQ, dK, dV
    return r


def check_kept_sets(gpu_idx, orc):
    """Kept lists must be equal except for swaps between candidates whose ORACLE pooled votes
    differ by less than 1e-5 relative.  Returns the number of swapped entries."""
    swaps = 0
    B, Hkv, n_kept = gpu_idx.shape
    for b in range(B):
        for h in range(Hkv):
            g, o = gpu_idx[b, h], orc.kept_idx[b, h]
            assert np.all(np.diff(g) > 0), "kept indices must be strictly ascending"
            if np.array_equal(g, o):
                continue
            only_g, only_o = np.setdiff1d(g, o), np.setdiff1d(o, g)
            assert only_g.size == only_o.size
            pg = np.sort(orc.pooled[b, h][only_g])
            po = np.sort(orc.pooled[b, h][only_o])
            rel = np.abs(pg - po) / np.maximum(np.maximum(pg, po), 1e-300)
            assert np.all(rel < SWAP_REL), f"unit ({b},{h}): kept sets differ beyond near-ties: rel {rel.max():.3e}"
            swaps += only_g.size
    return swaps


def assert_close_out(got, ref, what):
    err = np.abs(np.asarray(got, dtype=np.float64) - ref)
    assert np.isfinite(err).all(), f"{what}: non-finite values"
    assert err.max() <= OUT_MAX_ABS, f"{what}: max-abs {err.max():.3e}"
    assert err.mean() <= OUT_MEAN_ABS, f"{what}: mean-abs {err.mean():.3e}"
    return err.max(), err.mean()


def assert_close_lse(got, ref, what):
    got = np.asarray(got, dtype=np.float64)
    inf = np.isneginf(ref)
    assert np.array_equal(np.isneginf(got), inf), f"{what}: -inf pattern differs"
    err = np.abs(got[~inf] - ref[~inf])
    if err.size:
        assert err.max() <= LSE_ABS, f"{what}: max-abs {err.max():.3e}"
    return float(err.max()) if err.size else 0.0


def compare_compress(g, Q_obs, K, V, *, window, pool, budget, n_cal, orc=None):
    """Full comparison of a GPU compress result with the oracle.  Returns (oracle result used
    for downstream comparison, number of near-tie swaps)."""
    if orc is None:
        orc = oracle.compress(Q_obs, K, V, window=window, pool=pool, budget=budget, n_cal=n_cal, cap=g.cap)
    swaps = 0
    if budget < K.shape[2]:
        swaps = check_kept_sets(g.kept_idx, orc)
    else:
        np.testing.assert_array_equal(g.kept_idx, orc.kept_idx)
    ref = orc
    if swaps:
        ref = oracle.calibrate_given_indices(Q_obs, K, V, g.kept_idx, n_cal=n_cal, cap=g.cap)
    nk = g.n_kept
    np.testing.assert_array_equal(g.K_kept[:, :, :nk], ref.K_kept[:, :, :nk])
    np.testing.assert_array_equal(g.V_kept[:, :, :nk], ref.V_kept[:, :, :nk])
    np.testing.assert_array_equal(g.C_q, ref.C_q)
    assert_close_lse(g.LSE_c, ref.LSE_c, "LSE_c")
    assert_close_out(g.O_c, ref.O_c, "O_c")
    return ref, swaps


def decode_steps_compare(g, ref, q, kn, vn, *, theta1=0.7, theta2=0.85, steps=None, append=True):
    """Run decode steps on the GPU state `g.st` and on the oracle state `ref` (copied), and
    compare every step.  Discrete choices (row, gate) may differ only at near-ties, in which
    case the oracle is re-evaluated under the GPU's choice."""
    st, p = g.st, g.p
    p.theta1, p.theta2 = theta1, theta2
    T = q.shape[0] if steps is None else steps
    Kk, Vk = ref.K_kept.copy(), ref.V_kept.copy()
    kv_len = g.n_kept
    out = torch.empty((p.B, p.Hq, p.D), dtype=torch.bfloat16, device="cuda")
    lse = torch.empty((p.B, p.Hq), dtype=torch.float32, device="cuda")
    flags = torch.empty((p.B, p.Hq), dtype=torch.uint8, device="cuda")
    stats = dict(max_abs=0.0, mean_abs=0.0, lse=0.0, forced=0, applied=0, total=0)
    for t in range(T):
        dq = to_dev(q[t])
        dk = to_dev(kn[t]) if append else None
        dv = to_dev(vn[t]) if append else None
        cd.calidrop_decode(p, dq, dk, dv, st.K_kept, st.V_kept, kv_len, st.O_c, st.LSE_c, st.C_q, out, lse,
                           flags, st.ws_decode)
        torch.cuda.synchronize()
        off = cd.calidrop_decode_workspace_status_offset(p)
        assert int(st.ws_decode[off:off + 4].view(torch.int32).item()) == 0, "a wait of the decode kernel ran out"
        gout = wl.bf16_bits_to_f64(to_bits(out))
        gflags = flags.cpu().numpy()
        o = oracle.decode(q[t], kn[t] if append else None, vn[t] if append else None, Kk, Vk, kv_len,
                          ref.O_c, ref.LSE_c, ref.C_q, theta1=theta1, theta2=theta2)
        if not np.array_equal(gflags, o.flags):
            # allowed only at near-ties of the cosine similarity
            force_c = np.full((p.B, p.Hq), -1, dtype=np.int32)
            force_a = np.full((p.B, p.Hq), -1, dtype=np.int32)
            for b, hq in zip(*np.nonzero(gflags != o.flags)):
                rho = o.rho[b, hq]
                gc = int(gflags[b, hq] >> 2) if p.n_cal <= 64 else int(o.flags[b, hq] >> 2)
                oc = int(o.flags[b, hq] >> 2)
                if gc != oc:
                    assert abs(rho[gc] - rho[oc]) < 1e-4, "calibration row differs beyond a near-tie"
                    force_c[b, hq] = gc
                r = rho[gc]
                if (gflags[b, hq] & 1) != (o.flags[b, hq] & 1) and gc == oc:
                    assert abs(r - theta2) < 1e-3, "gate decision differs beyond a near-tie"
                if (gflags[b, hq] & 2) != (o.flags[b, hq] & 2) and gc == oc:
                    assert abs(r - theta1) < 1e-3, "recompute flag differs beyond a near-tie"
                force_a[b, hq] = int(gflags[b, hq] & 1)
                stats["forced"] += 1
            Kk2, Vk2 = Kk.copy(), Vk.copy()
            o = oracle.decode(q[t], kn[t] if append else None, vn[t] if append else None, Kk2, Vk2, kv_len,
                              ref.O_c, ref.LSE_c, ref.C_q, theta1=theta1, theta2=theta2,
                              force_c=force_c, force_apply=force_a)
            assert np.array_equal(gflags & 1, o.flags & 1)
        mx, mn = assert_close_out(gout, o.out, f"decode step {t}")
        le = assert_close_lse(lse.cpu().numpy(), o.lse, f"decode lse step {t}")
        stats["max_abs"] = max(stats["max_abs"], mx)
        stats["mean_abs"] = max(stats["mean_abs"], mn)
        stats["lse"] = max(stats["lse"], le)
        stats["applied"] += int((gflags & 1).sum())
        stats["total"] += gflags.size
        if append:
            kv_len += 1
    if append:
        nk = kv_len
        np.testing.assert_array_equal(to_bits(st.K_kept)[:, :, :nk], Kk[:, :, :nk])
        np.testing.assert_array_equal(to_bits(st.V_kept)[:, :, :nk], Vk[:, :, :nk])
    return stats
