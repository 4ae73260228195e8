"""Pins for the fp64 oracle: checks against what the paper and the mathematics fix.

Each test names the passage it pins.  None of them re-types the oracle's own formula:
they use library routines (torch softmax, numpy mean/cov/lstsq), special cases with a
known answer, the paper's alternative forms, and brute force on tiny shapes.
"""
import numpy as np
import pytest
import torch

TOL = 1e-10


def rand_case(seed, L, D, Dscale=1.0):
    g = np.random.default_rng(seed)
    q = g.standard_normal(D)
    r = g.standard_normal(D) * Dscale
    K = g.standard_normal((L, D))
    V = g.standard_normal((L, D))
    return q, r, K, V


def run_c(oracle, q, r, K, V, scale, L=None):
    """One (b=1, hq=1) call of the C oracle on float64 inputs."""
    T = K.shape[0]
    sl = None if L is None else np.array([L], dtype=np.int32)
    out, _ = oracle.decode_f64(q[None, None], r[None, None], K[None, None], V[None, None], sl, scale)
    return out[0, 0]


@pytest.mark.parametrize("L,D", [(1, 4), (7, 8), (64, 16), (300, 64)])
def test_zero_probe_is_softmax_attention(oracle, L, D):
    """rho = 0 recovers softmax attention exactly (Sec. 3.2, strong regularisation limit)."""
    q, r, K, V = rand_case(1, L, D)
    scale = 1.0 / np.sqrt(D)
    got = run_c(oracle, q, np.zeros(D), K, V, scale)
    p = torch.softmax(torch.from_numpy(K @ q * scale), dim=0)
    want = (p[None, :] @ torch.from_numpy(V))[0].numpy()
    np.testing.assert_allclose(got, want, rtol=0, atol=TOL)


def test_single_key_returns_its_value(oracle):
    """One key: p = 1 and the weighted covariance vanishes, so o = v_0 for any q, rho
    (definition of Sigma_KV under Eq. "parameterized_lla")."""
    q, r, K, V = rand_case(2, 1, 16, Dscale=5.0)
    np.testing.assert_allclose(run_c(oracle, q, r, K, V, 0.3), V[0], rtol=0, atol=TOL)
    # also through seqlens = 1 over a longer (ignored) cache
    q, r, K, V = rand_case(3, 9, 16)
    np.testing.assert_allclose(run_c(oracle, q, r, K, V, 0.3, L=1), V[0], rtol=0, atol=TOL)


def test_weights_sum_to_one(oracle):
    """The effective weights p_j (1 + tbar - t_j) sum to one (Sec. 4, score-pattern analysis),
    so a constant V comes back unchanged whatever the probe is."""
    q, r, K, _ = rand_case(4, 50, 8, Dscale=3.0)
    V = np.tile(np.array([[1.5, -2.0, 0.25, 7.0, 0, 1, 2, 3.0]]), (50, 1))
    np.testing.assert_allclose(run_c(oracle, q, r, K, V, 0.7), V[0], rtol=0, atol=1e-9)


def test_wide_bandwidth_limit_is_affine_linear_attention(oracle):
    """h -> infinity (scale = 0): o = vbar - S~ rho with uniform means, S~ = mean(v k^T) - vbar kbar^T
    (Sec. 3.2, wide bandwidth limit).  S~ is the biased cross-covariance block of numpy.cov."""
    q, r, K, V = rand_case(5, 40, 6)
    got = run_c(oracle, q, r, K, V, 0.0)
    D = K.shape[1]
    C = np.cov(np.concatenate([V, K], axis=1), rowvar=False, bias=True)
    S_tilde = C[:D, D:]                      # cov(v, k)
    want = V.mean(axis=0) - S_tilde @ r
    np.testing.assert_allclose(got, want, rtol=0, atol=TOL)


@pytest.mark.parametrize("seed,L,D", [(6, 5, 3), (7, 32, 8), (8, 200, 32)])
def test_three_forms_agree(oracle, seed, L, D):
    """Scoring form (C oracle) = covariance form with the explicit D x D Sigma_KV (brute force)
    = expanded form (Eq. "parallax_forward" both sides; Eq. "parallax_expand")."""
    q, r, K, V = rand_case(seed, L, D)
    scale = 1.0 / np.sqrt(D)
    a = run_c(oracle, q, r, K, V, scale)
    b = oracle.covariance_form(q, r, K, V, scale)
    c = oracle.expanded_form(q, r, K, V, scale)
    np.testing.assert_allclose(a, b, rtol=0, atol=TOL)
    np.testing.assert_allclose(a, c, rtol=0, atol=TOL)


@pytest.mark.parametrize("Bc", [1, 3, 16, 64, 1000])
def test_single_pass_walk_any_tile_size(oracle, Bc):
    """The single-pass tile walk of Sec. 3.3 (Algorithm 1) with any column-tile size reproduces the
    two-pass result."""
    q, r, K, V = rand_case(9, 150, 16)
    scale = 0.5
    want = run_c(oracle, q, r, K, V, scale)
    got = oracle.streaming_fold(q, r, K, V, scale, Bc)
    np.testing.assert_allclose(got, want, rtol=0, atol=TOL)


@pytest.mark.parametrize("cuts", [[0, 150], [0, 1, 150], [0, 40, 40, 97, 150], [0, 64, 128, 150]])
def test_split_merge_any_split_points(oracle, cuts):
    """Per-split partial states merged by log-sum-exp give the unsplit result, including an
    empty split (App. "Kernel Optimization Details", item 3)."""
    q, r, K, V = rand_case(10, 150, 16)
    scale = 0.5
    want = run_c(oracle, q, r, K, V, scale)
    states = [oracle.partial_state(q, r, K, V, scale, a, b) for a, b in zip(cuts[:-1], cuts[1:])]
    np.testing.assert_allclose(oracle.merge_partials(states), want, rtol=0, atol=TOL)


def test_exact_lla_link(oracle):
    """With rho = rho* (the exact local-linear solve) Parallax and LLA differ only by the boundary
    amplification: o_LLA = o_SA - (o_SA - o_PLX(rho*)) / (1 - tbar)  (Eq. "parameterized_lla").
    o_LLA itself comes from a generic least-squares solve of the weighted ridge local-linear
    regression with unpenalised intercept (Eq. "lla_forward").  Pins the sign and the orientation
    of the covariance term."""
    D, L, lam, h = 5, 30, 0.7, 2.0
    q, _, K, V = rand_case(11, L, D)
    scale = 1.0 / h
    w = np.exp(K @ q * scale)
    Z = K - q
    # textbook solve: minimise sum_j w_j |b + W z_j - v_j|^2 + lam |W|_F^2
    A = np.concatenate([np.sqrt(w)[:, None] * np.concatenate([np.ones((L, 1)), Z], axis=1),
                        np.sqrt(lam) * np.concatenate([np.zeros((D, 1)), np.eye(D)], axis=1)], axis=0)
    Y = np.concatenate([np.sqrt(w)[:, None] * V, np.zeros((D, D))], axis=0)
    o_lla = np.linalg.lstsq(A, Y, rcond=None)[0][0]
    # the paper's closed form of the same prediction
    mu = w @ Z
    Sigma = (w[:, None] * Z).T @ Z + lam * np.eye(D)
    rho_star = np.linalg.solve(Sigma, mu)
    o_lla_eq = ((w * (1 - Z @ rho_star)) @ V) / (w.sum() - mu @ rho_star)
    np.testing.assert_allclose(o_lla, o_lla_eq, rtol=0, atol=1e-9)
    p = w / w.sum()
    tbar = p @ (Z @ rho_star)
    assert 0.0 <= tbar < 1.0                                   # Proposition 1
    o_sa = run_c(oracle, q, np.zeros(D), K, V, scale)
    o_plx = run_c(oracle, q, rho_star, K, V, scale)
    np.testing.assert_allclose(o_lla, o_sa - (o_sa - o_plx) / (1.0 - tbar), rtol=0, atol=1e-9)


def test_invariances(oracle):
    """Consequences of the centred covariance and softmax shift-invariance: key permutation,
    affine dependence on rho, linearity in V, and independence of a key translation once the
    induced logit shift q.c is constant across keys (it always is)."""
    q, r, K, V = rand_case(12, 60, 8)
    scale = 0.4
    base = run_c(oracle, q, r, K, V, scale)
    perm = np.random.default_rng(0).permutation(60)
    np.testing.assert_allclose(run_c(oracle, q, r, K[perm], V[perm], scale), base, rtol=0, atol=TOL)
    c = np.random.default_rng(1).standard_normal(8)
    np.testing.assert_allclose(run_c(oracle, q, r, K + c, V, scale), base, rtol=0, atol=1e-9)
    r2 = np.random.default_rng(2).standard_normal(8)
    o0 = run_c(oracle, q, np.zeros(8), K, V, scale)
    o2 = run_c(oracle, q, r2, K, V, scale)
    mix = run_c(oracle, q, 2.0 * r - 3.0 * r2, K, V, scale)
    np.testing.assert_allclose(mix - o0, 2.0 * (base - o0) - 3.0 * (o2 - o0), rtol=0, atol=1e-9)
    V2 = np.random.default_rng(3).standard_normal((60, 8))
    np.testing.assert_allclose(run_c(oracle, q, r, K, 1.5 * V - V2, scale),
                               1.5 * base - run_c(oracle, q, r, K, V2, scale), rtol=0, atol=1e-9)


def test_probe_score_is_not_scaled(oracle):
    """Only S1 carries the softmax scale (Algorithm 1: S2 = R K^T has no factor s).  Hand-worked
    two-key example with uniform weights: k = (1, 3), v = (2, 6), rho = 0.5, scale = 0:
    t = (0.5, 1.5), tbar = 1, o = 0.5*(1.5)*2 + 0.5*(0.5)*6 = 3.  With scale = 0 any scaling of t
    by s would zero the correction and give 4 instead."""
    q = np.array([1.0])
    r = np.array([0.5])
    K = np.array([[1.0], [3.0]])
    V = np.array([[2.0], [6.0]])
    np.testing.assert_allclose(run_c(oracle, q, r, K, V, 0.0), [3.0], rtol=0, atol=TOL)
    # non-uniform weights: logits ln(3)*k_j*... use q = ln 3, k = (1, 0): p = (3/4, 1/4)
    q = np.array([np.log(3.0)])
    K = np.array([[1.0], [0.0]])
    V = np.array([[4.0], [8.0]])
    r = np.array([2.0])
    # t = (2, 0), tbar = 1.5, weights (3/4)(0.5) = 0.375 and (1/4)(2.5) = 0.625
    np.testing.assert_allclose(run_c(oracle, q, r, K, V, 1.0), [0.375 * 4 + 0.625 * 8], rtol=0, atol=TOL)


def test_gqa_mapping_seqlens_and_padding(oracle):
    """Batched call: consecutive query heads share a KV head, per-sequence lengths are honoured,
    rows past the length are never read into the result (NaN-poisoned), L = 0 gives zeros."""
    g = np.random.default_rng(13)
    B, Hq, Hkv, D, T = 3, 4, 2, 8, 20
    q = g.standard_normal((B, Hq, D))
    r = g.standard_normal((B, Hq, D))
    K = g.standard_normal((B, Hkv, T, D))
    V = g.standard_normal((B, Hkv, T, D))
    sl = np.array([20, 7, 0], dtype=np.int32)
    for b in range(B):
        K[b, :, sl[b]:] = np.nan
        V[b, :, sl[b]:] = np.nan
    out, _ = oracle.decode_f64(q, r, K, V, sl, 0.35)
    assert np.isfinite(out).all()
    np.testing.assert_array_equal(out[2], 0.0)
    for b in range(2):
        for hq in range(Hq):
            want = oracle.covariance_form(q[b, hq], r[b, hq], K[b, hq // 2, :sl[b]], V[b, hq // 2, :sl[b]], 0.35)
            np.testing.assert_allclose(out[b, hq], want, rtol=0, atol=TOL)


def test_bf16_entry_matches_f64_entry(oracle):
    """The bf16-bits entry converts exactly and then runs the same arithmetic."""
    from paper_2605_29157_b200 import workloads as wl
    cfg = wl.scaled(wl.CONFIGS["C1"], T_max=70)
    x = wl.make_inputs(cfg, "cpu")
    bits = {n: wl.bf16_bits(x[n]) for n in ("q", "r", "k", "v")}
    a, _ = oracle.decode_bf16(bits["q"], bits["r"], bits["k"], bits["v"], None, cfg.scale)
    f = {n: x[n].to(torch.float64).numpy() for n in ("q", "r", "k", "v")}
    b, _ = oracle.decode_f64(f["q"], f["r"], f["k"], f["v"], None, cfg.scale)
    np.testing.assert_array_equal(a, b)
    np.testing.assert_array_equal(oracle.bf16_bits_to_f64(bits["q"]), f["q"])


def test_threads_do_not_change_result(oracle):
    from paper_2605_29157_b200 import workloads as wl
    cfg = wl.scaled(wl.CONFIGS["C2"], B=2, T_max=33)
    x = wl.make_inputs(cfg, "cpu")
    bits = {n: wl.bf16_bits(x[n]) for n in ("q", "r", "k", "v")}
    a, n1 = oracle.decode_bf16(bits["q"], bits["r"], bits["k"], bits["v"], None, cfg.scale, threads=1)
    b, n2 = oracle.decode_bf16(bits["q"], bits["r"], bits["k"], bits["v"], None, cfg.scale, threads=0)
    assert n1 == 1 and n2 >= 1
    np.testing.assert_array_equal(a, b)


def test_stored_tiny_config_values(oracle):
    """The oracle still reproduces the values stored for the tiny configuration (written by
    tests/golden/make_golden.py from the oracle alone); guards against silent drift."""
    import hashlib
    from pathlib import Path
    from paper_2605_29157_b200 import workloads as wl
    lines = Path(__file__).with_name("golden").joinpath("c1_tiny_oracle.txt").read_text().splitlines()
    digest = [l.split()[2] for l in lines if l.startswith("# input_sha256")][0]
    want = np.array([float(l) for l in lines if not l.startswith("#")]).reshape(1, 2, 64)
    cfg = wl.CONFIGS["C1"]
    x = wl.make_inputs(cfg, "cpu")
    bits = {n: wl.bf16_bits(x[n]) for n in ("q", "r", "k", "v")}
    if hashlib.sha256(b"".join(bits[n].tobytes() for n in ("q", "r", "k", "v"))).hexdigest() != digest:
        pytest.skip("this torch build draws different seeded inputs than the stored file was made with")
    got, _ = oracle.decode_bf16(bits["q"], bits["r"], bits["k"], bits["v"], None, cfg.scale)
    np.testing.assert_allclose(got, want, rtol=0, atol=1e-13)


# ---------------------------------------------------------------------------------------------
# multi-token (causal) forward
# ---------------------------------------------------------------------------------------------
def _prefill_case(seed, B, Hq, Hkv, D, Lq, T):
    g = np.random.default_rng(seed)
    q = g.standard_normal((B, Hq, Lq, D))
    r = g.standard_normal((B, Hq, Lq, D))
    K = g.standard_normal((B, Hkv, T, D))
    V = g.standard_normal((B, Hkv, T, D))
    return q, r, K, V


def test_prefill_zero_probe_is_causal_softmax_attention(oracle):
    """rho = 0: causal softmax attention with the query block aligned to the END of the context,
    against torch's scaled_dot_product_attention with an explicit boolean mask (fp64)."""
    B, Hq, Hkv, D, Lq, T = 2, 4, 2, 8, 5, 12
    q, r, K, V = _prefill_case(20, B, Hq, Hkv, D, Lq, T)
    sl = np.array([12, 7], dtype=np.int32)
    got, _ = oracle.prefill_f64(q, np.zeros_like(r), K, V, sl, 0.3)
    for b in range(B):
        L = int(sl[b])
        mask = torch.zeros(Lq, L, dtype=torch.bool)
        for i in range(Lq):
            mask[i, :L - Lq + i + 1] = True
        kk = torch.from_numpy(K[b, :, :L]).repeat_interleave(Hq // Hkv, dim=0)
        vv = torch.from_numpy(V[b, :, :L]).repeat_interleave(Hq // Hkv, dim=0)
        want = torch.nn.functional.scaled_dot_product_attention(torch.from_numpy(q[b]), kk, vv, attn_mask=mask, scale=0.3)
        np.testing.assert_allclose(got[b], want.numpy(), rtol=0, atol=1e-10)


def test_prefill_rows_are_brute_force_covariance_form(oracle):
    """Every token row equals vbar - Sigma_KV rho over exactly its causal prefix (explicit D x D
    covariance), the first token of a fresh sequence returns v_0, a token with no key gives zeros."""
    B, Hq, Hkv, D, Lq, T = 2, 2, 1, 6, 4, 9
    q, r, K, V = _prefill_case(21, B, Hq, Hkv, D, Lq, T)
    sl = np.array([9, 3], dtype=np.int32)       # second sequence: fewer keys than query tokens
    got, _ = oracle.prefill_f64(q, r, K, V, sl, 0.45)
    for b in range(B):
        for h in range(Hq):
            for i in range(Lq):
                n = int(sl[b]) - Lq + i + 1
                if n <= 0:
                    np.testing.assert_array_equal(got[b, h, i], 0.0)
                    continue
                want = oracle.covariance_form(q[b, h, i], r[b, h, i], K[b, 0, :n], V[b, 0, :n], 0.45)
                np.testing.assert_allclose(got[b, h, i], want, rtol=0, atol=1e-10)
    q, r, K, V = _prefill_case(22, 1, 1, 1, 4, 3, 3)
    got, _ = oracle.prefill_f64(q, r, K, V, None, 1.0)
    np.testing.assert_allclose(got[0, 0, 0], V[0, 0, 0], rtol=0, atol=1e-12)


def test_prefill_single_token_is_the_decode_call(oracle):
    q, r, K, V = _prefill_case(23, 2, 4, 2, 8, 1, 10)
    a, _ = oracle.prefill_f64(q, r, K, V, None, 0.2)
    b, _ = oracle.decode_f64(q[:, :, 0], r[:, :, 0], K, V, None, 0.2)
    np.testing.assert_array_equal(a[:, :, 0], b)


# ---------------------------------------------------------------------------------------------
# upstream step: RMSNorm + rotary embedding
# ---------------------------------------------------------------------------------------------
def test_rmsnorm_matches_torch(oracle):
    g = np.random.default_rng(30)
    x, w = g.standard_normal((3, 5, 64)), g.standard_normal(64)
    want = torch.nn.functional.rms_norm(torch.from_numpy(x), (64,), torch.from_numpy(w), eps=1e-6).numpy()
    np.testing.assert_allclose(oracle.rmsnorm(x, w, 1e-6), want, rtol=0, atol=1e-12)


def test_rope_is_complex_rotation_and_relative(oracle):
    """Rotate-half RoPE = multiplying the complex numbers x_i + i x_{i+D/2} by exp(i pos theta^(-2i/D));
    it keeps norms, is the identity at position 0, and makes q.k depend on the position difference only."""
    g = np.random.default_rng(31)
    D, theta = 32, 1e6
    x, y = g.standard_normal(D), g.standard_normal(D)
    z = x[:D // 2] + 1j * x[D // 2:]
    rot = z * np.exp(1j * 1234 * theta ** (-2.0 * np.arange(D // 2) / D))
    got = oracle.rope(x, 1234, theta)
    np.testing.assert_allclose(got, np.concatenate([rot.real, rot.imag]), rtol=0, atol=1e-12)
    np.testing.assert_allclose(np.linalg.norm(got), np.linalg.norm(x), rtol=1e-13)
    np.testing.assert_allclose(oracle.rope(x, 0, theta), x, rtol=0, atol=0)
    a = oracle.rope(x, 5000, theta) @ oracle.rope(y, 4990, theta)
    b = oracle.rope(x, 17, theta) @ oracle.rope(y, 7, theta)
    np.testing.assert_allclose(a, b, rtol=0, atol=1e-9)


def test_prepare_step_composition(oracle):
    """The step applies the norm first, then the rotation at position seqlens-1; rho is rotated only on
    request; v passes through."""
    g = np.random.default_rng(32)
    B, Hq, Hkv, D = 2, 4, 2, 16
    qr, rr = g.standard_normal((B, Hq, D)), g.standard_normal((B, Hq, D))
    kr, vr = g.standard_normal((B, Hkv, D)), g.standard_normal((B, Hkv, D))
    wq, wr, wk = g.standard_normal(D), g.standard_normal(D), g.standard_normal(D)
    sl = np.array([9, 1])
    q, r, k, v = oracle.prepare_step(qr, rr, kr, vr, wq, wr, wk, sl, 1e-6, 1e6, False)
    np.testing.assert_array_equal(v, vr)
    np.testing.assert_allclose(r, oracle.rmsnorm(rr, wr, 1e-6), rtol=0, atol=0)
    np.testing.assert_allclose(q[1], oracle.rmsnorm(qr[1], wq, 1e-6), rtol=0, atol=1e-15)      # position 0
    np.testing.assert_allclose(q[0], oracle.rope(oracle.rmsnorm(qr[0], wq, 1e-6), 8, 1e6), rtol=0, atol=1e-15)
    _, r2, _, _ = oracle.prepare_step(qr, rr, kr, vr, wq, wr, wk, sl, 1e-6, 1e6, True)
    np.testing.assert_allclose(r2[0], oracle.rope(oracle.rmsnorm(rr[0], wr, 1e-6), 8, 1e6), rtol=0, atol=1e-15)
