"""The seeded input generator: determinism, bf16 rounding, and the statistics the recipe promises."""
import numpy as np
import torch

from paper_2507_19906_b200 import workload as wl


def test_bf16_rounding_matches_library_cast():
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.standard_normal(4096).astype(np.float32) * 10,
                        np.array([0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.3895314e38], np.float32)])
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    np.testing.assert_array_equal(wl.f32_to_bf16_bits(x), ref)
    back = wl.bf16_bits_to_f32(ref)
    np.testing.assert_array_equal(back, torch.from_numpy(x).to(torch.bfloat16).float().numpy())


def test_generator_is_deterministic_and_unit_addressable():
    cfg = wl.small_config(B=2, Hq=4, Hkv=2, L=64)
    K1, V1 = wl.gen_kv(cfg, threads=1)
    K2, V2 = wl.gen_kv(cfg, threads=4)
    np.testing.assert_array_equal(K1, K2)
    np.testing.assert_array_equal(V1, V2)
    k, v = wl.gen_kv_unit(cfg, 0, 1, 1)
    np.testing.assert_array_equal(k, K1[1, 1])
    np.testing.assert_array_equal(v, V1[1, 1])
    assert not np.array_equal(K1[0, 0], K1[1, 0])
    other = wl.gen_kv(cfg.scaled(seed=1))[0]
    assert not np.array_equal(other, K1)


def test_structure_sinks_heavy_keys_and_query_similarity():
    cfg = wl.CONFIGS[1]
    Q = wl.gen_q_obs(cfg)
    K, V = wl.gen_kv(cfg)
    q = wl.bf16_bits_to_f64(Q)[0]                      # [Hq, W, D]
    qn = q / np.linalg.norm(q, axis=-1, keepdims=True)
    adj = (qn[:, 1:] * qn[:, :-1]).sum(-1)
    assert 0.85 < adj.mean() < 0.95                    # nearby queries are similar
    k = wl.bf16_bits_to_f64(K)[0]
    norms = np.linalg.norm(k, axis=-1)                 # [Hkv, L]
    heavy = (norms > 30).sum(axis=1)
    assert np.all(heavy == cfg.n_heavy)
    assert np.all(norms[:, :cfg.n_sink].std(axis=1) < 1e-6)   # sink rows are identical
    assert np.all(norms[:, cfg.L - cfg.window:] < 30)  # no heavy key inside the window
    qd, kn, vn = wl.gen_decode_inputs(cfg, Q)
    qd = wl.bf16_bits_to_f64(qd)[:, 0]
    last = q[:, -1]
    cos = (qd * last).sum(-1) / (np.linalg.norm(qd, axis=-1) * np.linalg.norm(last, axis=-1))
    assert 0.86 < cos.mean() < 0.95                    # above theta2 = 0.85 on average
    assert qd.shape == (cfg.steps, cfg.Hq, cfg.D) and kn.shape == (cfg.steps, 1, cfg.Hkv, cfg.D)


def test_drifting_noise_schedule_and_rope():
    cfg = wl.CONFIGS[5]
    assert abs(cfg.sigma(0) - 0.1) < 1e-12 and abs(cfg.sigma(cfg.steps - 1) - 0.6) < 1e-12
    c4 = wl.CONFIGS[4].scaled(L=256, B=1, layers=1)
    k_rot, _ = wl.gen_kv_unit(c4, 0, 0, 0)
    k_raw, _ = wl.gen_kv_unit(c4.scaled(rope=False), 0, 0, 0)
    a, b = wl.bf16_bits_to_f64(k_rot), wl.bf16_bits_to_f64(k_raw)
    np.testing.assert_allclose(np.linalg.norm(a, axis=1), np.linalg.norm(b, axis=1), rtol=2e-2)
    np.testing.assert_array_equal(a[0], b[0])          # position 0 is not rotated
    assert not np.allclose(a[5], b[5])
