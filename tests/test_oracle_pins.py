"""Pins for the CPU oracle: every check here is against something the paper or
the mathematics fixes (closed forms, identities, brute force on tiny inputs,
numbers printed in the paper), never against the oracle's own formula retyped.
A few tests plant a plausible mistake in a copy of an oracle function and
check that a pin catches it."""
import math
import os

import numpy as np
import pytest

from oracle import slim_oracle as so
from paper_2503_05840_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _rand_case(seed, T, d, H, well_conditioned=True):
    g = np.random.default_rng(seed)
    X = g.standard_normal((T, d))
    W_Q = g.standard_normal((d, d)) / math.sqrt(d)
    W_V = g.standard_normal((d, d)) / math.sqrt(d)
    if well_conditioned:
        Qo, _ = np.linalg.qr(g.standard_normal((d, d)))
        W_K = Qo * g.uniform(0.5, 2.0, size=d)[None, :]
    else:
        W_K = g.standard_normal((d, d)) / math.sqrt(d)
    return X, W_Q, W_K, W_V


# ------------------------------------------------------------------ Eq. 6
def test_wkv_closed_form_for_orthogonal_times_diagonal():
    # W_K = Q diag(s)  =>  W_K^{-1} = diag(1/s) Q^T  exactly.
    _, W_K, W_V, Qo, s = synth.make_weights(48, 123)
    expect = (Qo.T @ W_V) / s[:, None]
    got = so.oracle_wkv(W_K, W_V)
    assert np.allclose(got, expect, rtol=1e-11, atol=1e-13)


def test_wkv_hand_inverted_2x2_and_3x3():
    W_K = np.array([[2.0, 1.0], [1.0, 1.0]])           # inverse [[1,-1],[-1,2]]
    W_V = np.array([[3.0, 0.0], [1.0, 2.0]])
    expect = np.array([[1.0, -1.0], [-1.0, 2.0]]) @ W_V
    assert np.allclose(so.oracle_wkv(W_K, W_V), expect, atol=1e-14)
    W_K3 = np.array([[1.0, 2.0, 0.0], [0.0, 1.0, 3.0], [0.0, 0.0, 1.0]])
    inv3 = np.array([[1.0, -2.0, 6.0], [0.0, 1.0, -3.0], [0.0, 0.0, 1.0]])
    W_V3 = np.arange(9.0).reshape(3, 3)
    assert np.allclose(so.oracle_wkv(W_K3, W_V3), inv3 @ W_V3, atol=1e-13)


def test_wkv_reconstructs_v_from_k():
    # Eq. 6: K W_KV = V, and the appendix-A check W_K W_KV ~ W_V (numpy allclose defaults).
    X, _, W_K, W_V = _rand_case(5, 9, 32, 4, well_conditioned=False)
    W_KV = so.oracle_wkv(W_K, W_V)
    assert np.allclose(W_K @ W_KV, W_V)
    assert np.allclose((X @ W_K) @ W_KV, X @ W_V, rtol=1e-8, atol=1e-9)
    assert np.allclose(np.linalg.inv(W_K) @ W_V, W_KV, rtol=1e-8, atol=1e-9)


def test_wkv_rejects_non_square():
    with pytest.raises(ValueError):
        so.oracle_wkv(np.zeros((4, 6)), np.zeros((4, 6)))


# ------------------------------------------------------------------ Eq. 7 == Eq. 2
@pytest.mark.parametrize("T,d,H,theta", [(1, 8, 2, 0.0), (7, 16, 4, 0.0), (33, 32, 4, 1.0e4),
                                         (64, 48, 6, 1.0e6), (130, 64, 2, 1.0e4)])
def test_slim_equals_vanilla_and_option1_equals_option2(T, d, H, theta):
    X, W_Q, W_K, W_V = _rand_case(100 + T, T, d, H)
    ref = so.oracle_vanilla(X, W_Q, W_K, W_V, H, theta)
    K = X @ W_K
    q = X[-1] @ W_Q
    W_KV = so.oracle_wkv(W_K, W_V)
    o2 = so.oracle_slim(q, K, W_KV, H, theta)
    o1 = so.oracle_slim_option1(q, K, W_KV, H, theta)
    scale = np.max(np.abs(ref))
    assert np.max(np.abs(o2 - ref)) <= 1e-11 * scale
    assert np.max(np.abs(o1 - ref)) <= 1e-11 * scale
    assert np.max(np.abs(o1 - o2)) <= 1e-11 * scale


def test_config0_shape_slim_equals_vanilla():
    cfg = synth.CONFIGS[0].scaled(context=300)
    L = synth.make_layer(cfg, synth.layer_seed(0, 0))
    X = L.X[0]
    ref = so.oracle_vanilla(X, L.W_Q, L.W_K, L.W_V, cfg.H, cfg.rope_theta)
    W_KV = so.oracle_wkv(L.W_K, L.W_V)
    got = so.oracle_slim(X[-1] @ L.W_Q, X @ L.W_K, W_KV, cfg.H, cfg.rope_theta)
    assert np.max(np.abs(got - ref)) <= 1e-11 * np.max(np.abs(ref))


# ------------------------------------------------------------------ T = 1, T = 2
@pytest.mark.parametrize("theta", [0.0, 1.0e4])
def test_single_key_returns_its_value_row(theta):
    X, W_Q, W_K, W_V = _rand_case(7, 1, 16, 4)
    W_KV = so.oracle_wkv(W_K, W_V)
    g = np.random.default_rng(0)
    for _ in range(3):
        q = g.standard_normal(16) * 5
        out = so.oracle_slim(q, X @ W_K, W_KV, 4, theta)
        assert np.allclose(out, (X @ W_V)[0], rtol=1e-10, atol=1e-12)


def test_two_keys_is_a_logistic_blend_hand_computed():
    # one head of width 2, no RoPE:  o = sig(a) v0 + (1 - sig(a)) v1,
    # a = (q.k0 - q.k1)/sqrt(2), all numbers chosen by hand.
    q = np.array([1.0, -2.0])
    K = np.array([[0.5, 0.25], [-1.0, 0.75]])
    W_KV = np.array([[2.0, 0.0], [1.0, -1.0]])
    V = np.array([[0.5 * 2 + 0.25 * 1, -0.25], [-2.0 + 0.75, -0.75]])
    s0 = (1.0 * 0.5 + -2.0 * 0.25) / math.sqrt(2.0)     # = 0
    s1 = (1.0 * -1.0 + -2.0 * 0.75) / math.sqrt(2.0)    # = -2.5/sqrt2
    w0 = 1.0 / (1.0 + math.exp(-(s0 - s1)))
    expect = w0 * V[0] + (1.0 - w0) * V[1]
    assert np.allclose(so.oracle_slim(q, K, W_KV, 1, 0.0), expect, rtol=1e-13)
    assert np.allclose(so.oracle_slim_option1(q, K, W_KV, 1, 0.0), expect, rtol=1e-13)


def test_two_keys_with_rope_hand_rotation_2d():
    # d_k = 2: one frequency theta_0 = 1, so key t is rotated by angle t and the
    # query (position 1) by angle 1, with the appendix's sign:
    #   y1 = x1 cos + x2 sin ; y2 = -x1 sin + x2 cos
    theta = 10000.0
    q = np.array([0.3, -1.1])
    K = np.array([[1.5, 0.2], [-0.4, 0.9]])
    W_KV = np.array([[1.0, 2.0], [3.0, 4.0]])
    c1, s1 = math.cos(1.0), math.sin(1.0)
    qr = np.array([q[0] * c1 + q[1] * s1, -q[0] * s1 + q[1] * c1])
    k0r = K[0]                                              # angle 0
    k1r = np.array([K[1][0] * c1 + K[1][1] * s1, -K[1][0] * s1 + K[1][1] * c1])
    z0 = float(qr @ k0r) / math.sqrt(2.0)
    z1 = float(qr @ k1r) / math.sqrt(2.0)
    w0 = math.exp(z0) / (math.exp(z0) + math.exp(z1))
    V = K @ W_KV
    expect = w0 * V[0] + (1 - w0) * V[1]
    assert np.allclose(so.oracle_slim(q, K, W_KV, 1, theta), expect, rtol=1e-13)


def test_rope_frequency_schedule_and_pairing_dk4():
    # d_k = 4, theta = 10000: theta_0 = 1, theta_1 = 10000^(-1/2) = 0.01;
    # element 0 pairs with 2, element 1 pairs with 3.
    x = np.array([1.0, 2.0, 3.0, 4.0])
    m = 3
    y = so.rope_encode(x, m, 10000.0)
    c0, s0 = math.cos(3.0), math.sin(3.0)
    c1, s1 = math.cos(0.03), math.sin(0.03)
    expect = np.array([1 * c0 + 3 * s0, 2 * c1 + 4 * s1, -1 * s0 + 3 * c0, -2 * s1 + 4 * c1])
    assert np.allclose(y, expect, rtol=1e-14)
    assert np.allclose(so.rope_frequencies(4, 10000.0), [1.0, 0.01], rtol=1e-14)


# ------------------------------------------------------------------ uniform keys
@pytest.mark.parametrize("theta", [0.0, 1.0e4])
def test_identical_keys_return_their_value(theta):
    g = np.random.default_rng(3)
    d, H, T = 24, 3, 50
    _, W_K, W_V, _, _ = synth.make_weights(d, 9)
    k = g.standard_normal(d)
    K = np.tile(k, (T, 1))
    W_KV = so.oracle_wkv(W_K, W_V)
    out = so.oracle_slim(g.standard_normal(d), K, W_KV, H, theta)
    assert np.allclose(out, k @ W_KV, rtol=1e-10, atol=1e-12)


# ------------------------------------------------------------------ softmax
def test_softmax_rows_sum_to_one_and_shift_invariant():
    g = np.random.default_rng(1)
    z = g.standard_normal((5, 40)) * 30
    p = so.softmax(z)
    assert np.allclose(p.sum(axis=-1), 1.0, rtol=1e-14)
    assert np.allclose(so.softmax(z + 123.456), p, rtol=1e-10)
    assert np.allclose(so.softmax(np.array([0.0, math.log(3.0)])), [0.25, 0.75], rtol=1e-14)
    assert np.all(np.isfinite(so.softmax(np.array([1e4, -1e4, 0.0]))))


def test_attention_weights_sum_to_one():
    g = np.random.default_rng(2)
    w = so.attention_weights(g.standard_normal(8), g.standard_normal((19, 8)), 1.0e4)
    assert abs(w.sum() - 1.0) < 1e-14 and np.all(w > 0)


# ------------------------------------------------------------------ RoPE
def test_rope_decode_inverts_encode_and_preserves_norm():
    g = np.random.default_rng(4)
    x = g.standard_normal((11, 3, 16))
    pos = np.arange(11)[:, None] * 977
    y = so.rope_encode(x, pos, 1.0e6)
    assert np.allclose(so.rope_decode(y, pos, 1.0e6), x, rtol=1e-12, atol=1e-13)
    assert np.allclose(np.linalg.norm(y, axis=-1), np.linalg.norm(x, axis=-1), rtol=1e-13)
    assert not np.allclose(y[1:], x[1:])


def test_rope_scores_depend_on_relative_position_only():
    g = np.random.default_rng(5)
    q, k = g.standard_normal(32), g.standard_normal(32)
    a = so.rope_encode(q, 100, 1.0e4) @ so.rope_encode(k, 37, 1.0e4)
    b = so.rope_encode(q, 100 + 555, 1.0e4) @ so.rope_encode(k, 37 + 555, 1.0e4)
    c = so.rope_encode(q, 101, 1.0e4) @ so.rope_encode(k, 37, 1.0e4)
    assert abs(a - b) < 1e-10
    assert abs(a - c) > 1e-3


def test_rope_theta_zero_is_identity_and_position_zero_is_identity():
    x = np.arange(8.0)
    assert np.array_equal(so.rope_encode(x, 5, 0.0), x)
    assert np.allclose(so.rope_encode(x, 0, 1.0e4), x)


def test_rotation_sign_is_a_real_convention():
    # score = cos(D)(q1 k1 + q2 k2) + sin(D)(q1 k2 - q2 k1) with D the relative
    # angle: turning both vectors the other way flips the sine term, so the
    # printed sign has to be followed literally (it is not a free choice).
    q, k = np.array([1.0, 0.0]), np.array([0.0, 1.0])
    enc = so.rope_encode(q, 1, 10000.0) @ so.rope_encode(k, 0, 10000.0)
    dec = so.rope_decode(q, 1, 10000.0) @ so.rope_decode(k, 0, 10000.0)
    # query rotated by -1 rad (printed sign): (cos1, -sin1) . (0, 1) = -sin 1
    assert abs(enc - (-math.sin(1.0))) < 1e-15
    assert abs(dec - (+math.sin(1.0))) < 1e-15


def test_key_bias_cancels_in_the_attention_weights_without_rope():
    # appendix "Support for bias": a constant added to every key shifts all
    # softmax arguments of one query by the same amount.
    g = np.random.default_rng(6)
    q, K, c = g.standard_normal(8), g.standard_normal((15, 8)), g.standard_normal(8)
    assert np.allclose(so.attention_weights(q, K + c, 0.0), so.attention_weights(q, K, 0.0), rtol=1e-10)


# ------------------------------------------------------------------ brute force + OP count
@pytest.mark.parametrize("T,d,H,theta", [(5, 8, 2, 0.0), (6, 12, 3, 1.0e4), (9, 8, 1, 1.0e6)])
def test_scalar_loops_match_vectorised_and_count_macs(T, d, H, theta):
    X, W_Q, W_K, W_V = _rand_case(50 + T, T, d, H)
    K, q = X @ W_K, X[-1] @ W_Q
    W_KV = so.oracle_wkv(W_K, W_V)
    out, macs = so.oracle_slim_loops(q, K, W_KV, H, theta)
    assert np.allclose(out, so.oracle_slim(q, K, W_KV, H, theta), rtol=1e-11, atol=1e-13)
    # appendix "MHA complexity": 2 n d (h+1) OPs = n d (h+1) multiply-accumulates
    assert macs == T * d * (H + 1)


# ------------------------------------------------------------------ ragged batch
def test_batch_wrapper_masks_rows_beyond_length_and_zero_length():
    g = np.random.default_rng(8)
    d, H, B, Tc = 16, 2, 3, 12
    _, W_K, W_V, _, _ = synth.make_weights(d, 1)
    W_KV = so.oracle_wkv(W_K, W_V)
    K = g.standard_normal((B, Tc, d))
    q = g.standard_normal((B, d))
    lengths = np.array([12, 0, 5])
    K2 = K.copy()
    K2[2, 5:] = np.nan
    out = so.oracle_slim_batch(q, K2, lengths, W_KV, H, 1.0e4)
    assert np.all(out[1] == 0)
    assert np.allclose(out[0], so.oracle_slim(q[0], K[0], W_KV, H, 1.0e4))
    assert np.allclose(out[2], so.oracle_slim(q[2], K[2, :5], W_KV, H, 1.0e4))


# ------------------------------------------------------------------ planted mistakes
def _slim_with(q, K, W_KV, H, theta, *, scale=None, transpose=False, q_pos_shift=0, full_d=True):
    """oracle_slim with one deliberate defect, to show the pins notice it."""
    T, d = K.shape
    d_k = d // H
    out = np.empty(d)
    for i in range(H):
        sl = slice(i * d_k, (i + 1) * d_k)
        qr = so.rope_encode(q[sl], T - 1 + q_pos_shift, theta)
        Kr = so.rope_encode(K[:, sl], np.arange(T), theta)
        s = so.softmax(Kr @ qr / (math.sqrt(d_k) if scale is None else scale))
        W = W_KV.T if transpose else W_KV
        if full_d:
            out[sl] = (s @ K) @ W[:, sl]
        else:                       # wrongly uses only the head's own key slice
            out[sl] = (s @ K[:, sl]) @ W[sl, sl]
    return out


def test_pins_catch_planted_mistakes():
    T, d, H, theta = 40, 16, 2, 1.0e4
    X, W_Q, W_K, W_V = _rand_case(77, T, d, H)
    K, q = X @ W_K, X[-1] @ W_Q
    W_KV = so.oracle_wkv(W_K, W_V)
    ref = so.oracle_vanilla(X, W_Q, W_K, W_V, H, theta)
    tol = 1e-9 * np.max(np.abs(ref))
    assert np.max(np.abs(_slim_with(q, K, W_KV, H, theta) - ref)) < tol          # sane copy passes
    assert np.max(np.abs(_slim_with(q, K, W_KV, H, theta, transpose=True) - ref)) > 1e3 * tol
    assert np.max(np.abs(_slim_with(q, K, W_KV, H, theta, q_pos_shift=1) - ref)) > 1e3 * tol
    assert np.max(np.abs(_slim_with(q, K, W_KV, H, theta, full_d=False) - ref)) > 1e3 * tol
    # a dropped 1/sqrt(d_k) is caught by the hand-computed two-key blend:
    q2 = np.array([1.0, -2.0]); K2 = np.array([[0.5, 0.25], [-1.0, 0.75]])
    W2 = np.array([[2.0, 0.0], [1.0, -1.0]])
    good = so.oracle_slim(q2, K2, W2, 1, 0.0)
    bad = _slim_with(q2, K2, W2, 1, 0.0, scale=1.0)
    assert np.max(np.abs(good - bad)) > 1e-3


# ------------------------------------------------------------------ numbers printed in the paper
def _rows(name):
    with open(os.path.join(GOLD, name)) as f:
        return [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]


def test_kcache_accounting_matches_whisper_table():
    for model, d, layers, cross, self_, base, opt1 in _rows("whisper_cache_sizes.txt"):
        d, layers = int(d), int(layers)
        cross_k = synth.kcache_values(d, layers, 1500)
        self_k = synth.kcache_values(d, layers, 448)
        assert abs(2 * cross_k / 1e6 - float(cross)) <= 0.051
        assert abs(2 * self_k / 1e6 - float(self_)) <= 0.051
        assert abs(2 * (cross_k + self_k) / 1e6 - float(base)) <= 0.051
        assert abs((cross_k + self_k) / 1e6 - float(opt1)) <= 0.051   # K-cache only = half


def test_kcache_accounting_matches_table1():
    for model, d, layers, ctx, printed in _rows("table1_context_memory.txt"):
        kv = 2 * synth.kcache_values(int(d), int(layers), int(ctx))
        assert abs(kv - float(printed)) / float(printed) < 0.03


# ------------------------------------------------------------------ error norms
def test_error_norms():
    ref = np.array([3.0, -4.0, 0.0, 0.0])            # RMS = 2.5
    got = ref + np.array([0.0, 0.0, 0.25, 0.0])
    assert abs(so.err_rms_norm(got, ref) - 0.1) < 1e-15
    assert abs(so.err_fp32_norm(got, ref) - 0.1) < 1e-15
    got2 = ref + np.array([0.3, 0.0, 0.0, 0.0])
    assert abs(so.err_fp32_norm(got2, ref) - 0.1) < 1e-15   # relative to |ref_i| = 3


# ---- non-square projections, Option 1 (right inverse) -----------------------
def test_right_inverse_hand_example_1x2():
    # W_K = [3 4]: W_K W_K^T = 25, right inverse = [3 4]^T / 25; W_V = [1 2]
    W_K = np.array([[3.0, 4.0]]); W_V = np.array([[1.0, 2.0]])
    W_KV = so.oracle_wkv_right_inverse(W_K, W_V)
    assert np.allclose(W_KV, np.array([[3.0, 6.0], [4.0, 8.0]]) / 25.0, rtol=0, atol=1e-15)
    for x in (1.0, -2.5):
        assert np.allclose((x * W_K) @ W_KV, x * W_V)          # K W_KV = V


def test_right_inverse_properties_and_closed_form():
    from paper_2503_05840_b200 import synth
    d, e = 6, 16
    W_Q, W_K, W_V, Qrows, s = synth.make_weights_nonsquare(d, e, 11)
    W_KV = so.oracle_wkv_right_inverse(W_K, W_V)
    assert W_KV.shape == (e, e)
    assert np.allclose(W_K @ W_KV, W_V, rtol=1e-12, atol=1e-13)                   # W_K W_K^{-1} W_V = W_V
    assert np.allclose(W_KV, Qrows.T @ (W_V / s[:, None]), rtol=1e-11, atol=1e-13)  # rows of W_K are s_i q_i
    Rinv = so.oracle_wkv_right_inverse(W_K, np.eye(d) @ W_K)                      # W_K^{-1} W_K: projector on the row space
    assert np.allclose(Rinv, Rinv.T, atol=1e-12) and np.allclose(Rinv @ Rinv, Rinv, atol=1e-12)
    assert abs(np.trace(Rinv) - d) < 1e-10
    X = np.random.default_rng(0).standard_normal((9, d))
    assert np.allclose((X @ W_K) @ W_KV, X @ W_V, rtol=1e-11, atol=1e-12)          # V from K for any input


def test_right_inverse_reduces_to_the_inverse_for_square_weights():
    g = np.random.default_rng(3)
    W_K = g.standard_normal((7, 7)) + 3 * np.eye(7); W_V = g.standard_normal((7, 7))
    assert np.allclose(so.oracle_wkv_right_inverse(W_K, W_V), so.oracle_wkv(W_K, W_V), rtol=1e-9, atol=1e-11)


def test_slim_equals_vanilla_with_nonsquare_projections():
    from paper_2503_05840_b200 import synth
    d, e, H, T = 6, 16, 2, 13
    W_Q, W_K, W_V, _, _ = synth.make_weights_nonsquare(d, e, 5)
    X = np.random.default_rng(1).standard_normal((T, d))
    for theta in (0.0, 1.0e4):
        van = so.oracle_vanilla(X, W_Q, W_K, W_V, H, theta)
        slim = so.oracle_slim(X[-1] @ W_Q, X @ W_K, so.oracle_wkv_right_inverse(W_K, W_V), H, theta)
        assert van.shape == (e,)
        assert np.allclose(slim, van, rtol=1e-10, atol=1e-12)


# ---- X-cache / E-cache scheme (non-square Option 2, encoder-decoder Option 2) ----
def test_xcache_equals_vanilla_square_and_nonsquare_with_query_bias():
    from paper_2503_05840_b200 import synth
    g = np.random.default_rng(4)
    for d, e, H, T in ((8, 8, 2, 11), (6, 16, 4, 9)):
        if d == e:
            W_Q, W_K, W_V, _, _ = synth.make_weights(d, 3)
        else:
            W_Q, W_K, W_V, _, _ = synth.make_weights_nonsquare(d, e, 3)
        X = g.standard_normal((T, d))
        bias = g.standard_normal(e)
        q = X[-1] @ W_Q + bias
        van = so.oracle_vanilla(X, W_Q, W_K, W_V, H, 0.0, q=q)       # explicit K and V, same biased query
        xc = so.oracle_xcache(q, X, W_K, W_V, H)
        assert np.allclose(xc, van, rtol=1e-11, atol=1e-13)


def test_xcache_single_token_and_identical_rows():
    g = np.random.default_rng(6)
    d, H = 8, 2
    W_K = g.standard_normal((d, d)); W_V = g.standard_normal((d, d))
    x0 = g.standard_normal(d); q = g.standard_normal(d)
    assert np.allclose(so.oracle_xcache(q, x0[None, :], W_K, W_V, H), x0 @ W_V)          # T = 1: the value row
    X = np.tile(x0, (7, 1))
    assert np.allclose(so.oracle_xcache(q, X, W_K, W_V, H), x0 @ W_V)                    # uniform softmax


def test_xcache_two_tokens_closed_form():
    # one head, d = 2: scores a_t = (q W_K^T) . x_t / sqrt(2); output = sigma(a0 - a1) v0 + (1 - sigma) v1
    W_K = np.array([[1.0, 2.0], [0.5, -1.0]]); W_V = np.array([[2.0, 0.0], [1.0, 3.0]])
    X = np.array([[1.0, 0.0], [0.0, 2.0]]); q = np.array([0.3, -0.7])
    qt = q @ W_K.T
    a = X @ qt / np.sqrt(2.0)
    sig = 1.0 / (1.0 + np.exp(-(a[0] - a[1])))
    want = sig * (X[0] @ W_V) + (1 - sig) * (X[1] @ W_V)
    assert np.allclose(so.oracle_xcache(q, X, W_K, W_V, 1), want, rtol=1e-13)


# ---- head -> column-block mapping for more than one head (Eq. 4 / 5 / 2: head i owns the
# ---- i-th block of d_k consecutive columns of Q, K, V) -------------------------------------
def _two_head_hand_case():
    """d = 4, H = 2 (d_k = 2), T = 2, no RoPE; every number typed in.  With W_Q = W_K = I the keys
    are the inputs and q is the last input row.  Head 0 (columns 0, 1) sees two equal scores
    (q.k0 = q.k1 = 1), so it blends the values 1/2 : 1/2.  Head 1 (columns 2, 3) sees
    q.(k1 - k0) / sqrt(2) = sqrt(2) (sqrt(2) - c) / sqrt(2) = ln 3 with c = sqrt(2) - ln 3, so it
    blends 1/4 : 3/4.  A head that took columns (0, 2) or (1, 3) instead would get other scores."""
    r2, c = math.sqrt(2.0), math.sqrt(2.0) - math.log(3.0)
    X = np.array([[1.0, 5.0, c, 7.0],
                  [1.0, 0.0, r2, 0.0]])
    W_V = np.array([[1.0, 2.0, 0.0, 1.0],
                    [0.0, 1.0, 1.0, 0.0],
                    [2.0, 0.0, 1.0, 1.0],
                    [1.0, 1.0, 0.0, 2.0]])
    # value rows by hand: v0 = x0 W_V, v1 = x1 W_V
    v0 = np.array([8.0 + 2.0 * c, 14.0, 5.0 + c, 15.0 + c])
    v1 = np.array([1.0 + 2.0 * r2, 2.0, r2, 1.0 + r2])
    expect = np.array([0.5 * v0[0] + 0.5 * v1[0], 0.5 * v0[1] + 0.5 * v1[1],       # head 0: columns 0, 1
                       0.25 * v0[2] + 0.75 * v1[2], 0.25 * v0[3] + 0.75 * v1[3]])  # head 1: columns 2, 3
    return X, W_V, expect


def test_two_heads_hand_computed_column_blocks():
    X, W_V, expect = _two_head_hand_case()
    I4 = np.eye(4)
    assert np.allclose(so.oracle_vanilla(X, I4, I4, W_V, 2, 0.0), expect, rtol=1e-13)
    # slim attention on scaled keys: W_K = diag(2, 1, 1, 1/2), W_Q = W_K^{-1} (every q.k product is
    # unchanged), and W_KV = W_K^{-1} W_V typed row by row
    D = np.array([2.0, 1.0, 1.0, 0.5])
    K = X * D[None, :]
    q = X[1] / D
    W_KV = np.array([[0.5, 1.0, 0.0, 0.5],
                     [0.0, 1.0, 1.0, 0.0],
                     [2.0, 0.0, 1.0, 1.0],
                     [2.0, 2.0, 0.0, 4.0]])
    assert np.allclose(so.oracle_slim(q, K, W_KV, 2, 0.0), expect, rtol=1e-13)
    assert np.allclose(so.oracle_slim_option1(q, K, W_KV, 2, 0.0), expect, rtol=1e-13)
    assert np.allclose(so.oracle_slim_loops(q, K, W_KV, 2, 0.0)[0], expect, rtol=1e-13)
    assert np.allclose(so.oracle_slim_batch(q[None, :], K[None, :, :], [2], W_KV, 2, 0.0)[0], expect, rtol=1e-13)
    # X-cache scheme with the same scaled projections: q = x_n W_Q, cache holds X
    assert np.allclose(so.oracle_xcache(q, X, np.diag(D), W_V, 2), expect, rtol=1e-13)


def test_two_head_pin_catches_a_strided_head_slice():
    # the same arithmetic with head i = columns i, i + H, ... (a plausible mistake that every
    # single-head pin and the slim == vanilla identity would let through)
    X, W_V, expect = _two_head_hand_case()
    V = X @ W_V
    out = np.empty(4)
    for i in range(2):
        cols = [i, i + 2]
        s = so.softmax(X[:, cols] @ X[1, cols] / math.sqrt(2.0))
        out[cols] = s @ V[:, cols]
    assert np.max(np.abs(out - expect)) > 1e-2


# ---- rotated-key cache with skipped scores (sparsity appendix + RoPE appendix Option 2) -------------
def _rotated(K, H, theta):
    T, d = K.shape
    return so.rope_encode(K.reshape(T, H, d // H), np.arange(T)[:, None], theta).reshape(T, d)


def test_rotated_cache_hand_case_one_row_skipped():
    # one head of width 2, theta = 10000 (one frequency, angle = position): key 1 is stored rotated by
    # 1 rad (typed with cos 1, sin 1), key 0 at position 0 is stored as it is.  q is chosen so that the
    # rotated query is (1, 0): q = decode_1((1, 0)) = (cos 1, sin 1).  Scores: z0 = k0r[0]/sqrt 2,
    # z1 = k1r[0]/sqrt 2 with k0r = (0, 3), k1r = (sqrt 2 ln 9, 5)  =>  z1 - z0 = ln 9, s = (0.1, 0.9).
    c1, s1 = math.cos(1.0), math.sin(1.0)
    q = np.array([c1, s1])
    K_rot = np.array([[0.0, 3.0], [math.sqrt(2.0) * math.log(9.0), 5.0]])
    W_KV = np.array([[1.0, 2.0], [3.0, 4.0]])
    # raw keys by the decoding formulas: x1 = y1 cos - y2 sin, x2 = y1 sin + y2 cos
    k0 = K_rot[0]
    k1 = np.array([K_rot[1][0] * c1 - K_rot[1][1] * s1, K_rot[1][0] * s1 + K_rot[1][1] * c1])
    v0, v1 = k0 @ W_KV, k1 @ W_KV
    full, kept = so.oracle_rotated_cache(q, K_rot, W_KV, 1, 10000.0, threshold=0.0)
    assert kept[0] == 2 and np.allclose(full, 0.1 * v0 + 0.9 * v1, rtol=1e-12)
    cut, kept = so.oracle_rotated_cache(q, K_rot, W_KV, 1, 10000.0, threshold=0.5)
    assert kept[0] == 1 and np.allclose(cut, 0.9 * v1, rtol=1e-12)          # skipped, not renormalised
    none, kept = so.oracle_rotated_cache(q, K_rot, W_KV, 1, 10000.0, threshold=0.95)
    assert kept[0] == 0 and np.all(none == 0)


@pytest.mark.parametrize("theta", [0.0, 1.0e4, 1.0e6])
def test_rotated_cache_without_skipping_is_vanilla_attention(theta):
    T, d, H = 37, 32, 4
    X, W_Q, W_K, W_V = _rand_case(31, T, d, H)
    K = X @ W_K
    out, kept = so.oracle_rotated_cache(X[-1] @ W_Q, _rotated(K, H, theta), so.oracle_wkv(W_K, W_V), H, theta, threshold=-1.0)
    ref = so.oracle_vanilla(X, W_Q, W_K, W_V, H, theta)
    assert np.all(kept == T)
    assert np.max(np.abs(out - ref)) <= 1e-10 * np.max(np.abs(ref))


def test_rotated_cache_error_is_bounded_by_the_skipped_mass_and_work_shrinks():
    # peaked attention: a few keys aligned with the query.  For every head the error of the skipped
    # sum is at most (skipped probability mass) x (largest value row norm), and the rows decoded are
    # exactly those above the threshold (complexity factor 1 / (1 - S) of the sparsity appendix).
    g = np.random.default_rng(12)
    T, d, H, theta = 200, 16, 2, 1.0e4
    X, W_Q, W_K, W_V = _rand_case(32, T, d, H)
    K = X @ W_K
    q = X[-1] @ W_Q * 6.0
    W_KV = so.oracle_wkv(W_K, W_V)
    K_rot = _rotated(K, H, theta)
    exact = so.oracle_slim(q, K, W_KV, H, theta)
    V = K @ W_KV
    d_k = d // H
    for thr in (1e-4, 1e-2, 0.2):
        out, kept = so.oracle_rotated_cache(q, K_rot, W_KV, H, theta, thr)
        for i in range(H):
            sl = slice(i * d_k, (i + 1) * d_k)
            s = so.attention_weights(q[sl], K[:, sl], theta)
            assert kept[i] == int(np.sum(s > thr))
            skipped = float(np.sum(s[s <= thr]))
            bound = skipped * np.max(np.linalg.norm(V[:, sl], axis=1))
            assert np.linalg.norm(out[sl] - exact[sl]) <= bound + 1e-12
    # S = 0.8 exactly: ten keys, two of them carry everything above the threshold
    qh = np.array([1.0, 0.0]); Kh = np.zeros((10, 2)); Kh[[3, 7], 0] = 20.0
    _, kept = so.oracle_rotated_cache(qh, Kh, np.eye(2), 1, 0.0, threshold=1e-3)
    assert kept[0] == 2                                  # 1 / (1 - 0.8) = 5 times fewer rows in the weighted sum


def test_rotated_cache_pin_catches_a_missing_decode():
    # the same sum with the kept rows used as stored (still rotated) must differ
    T, d, H, theta = 20, 8, 2, 1.0e4
    X, W_Q, W_K, W_V = _rand_case(33, T, d, H)
    K = X @ W_K; q = X[-1] @ W_Q; W_KV = so.oracle_wkv(W_K, W_V)
    K_rot = _rotated(K, H, theta)
    good, _ = so.oracle_rotated_cache(q, K_rot, W_KV, H, theta, -1.0)
    bad = so.oracle_slim(q, K, W_KV, H, theta) * 0
    d_k = d // H
    for i in range(H):
        sl = slice(i * d_k, (i + 1) * d_k)
        s = so.attention_weights(q[sl], K[:, sl], theta)
        bad[sl] = (s @ K_rot) @ W_KV[:, sl]
    assert np.max(np.abs(good - bad)) > 1e-3 * np.max(np.abs(good))


def test_prompt_values_from_keys_are_the_vanilla_values():
    # Fig. 3(a) / Eq. 6: V = K W_KV equals X W_V (Eq. 5) for every prompt row, and one row by hand
    X, _, W_K, W_V = _rand_case(40, 11, 12, 3, well_conditioned=False)
    V = so.oracle_prompt_values(X @ W_K, so.oracle_wkv(W_K, W_V))
    assert np.allclose(V, X @ W_V, rtol=1e-9, atol=1e-11)
    K = np.array([[1.0, 2.0], [0.0, -1.0]]); W = np.array([[3.0, 1.0], [2.0, 0.5]])
    assert np.array_equal(so.oracle_prompt_values(K, W), np.array([[7.0, 2.0], [-2.0, -0.5]]))


# ---- 8-bit K-cache: the E4M3 format and the per-(row, head) power-of-two exponent -----------------
def test_e4m3_table_and_rounding_against_the_published_format():
    tab = so.e4m3_decode_table()
    # values fixed by the OCP FP8 definition: largest finite 448 = 0x7e, 1.0 = 0x38, smallest normal
    # 2^-6 = 0x08, smallest subnormal 2^-9 = 0x01, 0x7f and 0xff are NaN, negative half mirrors
    assert tab[0x7E] == 448.0 and tab[0x38] == 1.0 and tab[0x08] == 2.0 ** -6 and tab[0x01] == 2.0 ** -9
    assert tab[0x00] == 0.0 and np.isnan(tab[0x7F]) and np.isnan(tab[0xFF]) and tab[0xB8] == -1.0
    assert tab[0x3C] == 1.5 and tab[0x40] == 2.0 and tab[0x47] == 3.75
    assert np.all(np.diff(tab[:0x7F]) > 0)                       # codes are ordered like their values
    enc = so.e4m3_encode
    assert list(enc(np.array([448.0, 1.0, 1.5, -1.0, 0.0, 1e9, -1e9]))) == [0x7E, 0x38, 0x3C, 0xB8, 0x00, 0x7E, 0xFE]
    # every finite code survives decode -> encode; midpoints go to the even code (hand: 1.0625 is halfway
    # between 1.0 = 0x38 and 1.125 = 0x39 -> 0x38; 1.1875 halfway between 0x39 and 0x3a -> 0x3a)
    finite = [c for c in range(256) if not np.isnan(tab[c]) and c != 0x80]
    assert all(int(enc(np.array([tab[c]]))[0]) == c for c in finite)
    assert list(enc(np.array([1.0625, 1.1875, 1.06, 1.07, 2.0 ** -10, 1.5 * 2.0 ** -9]))) == [0x38, 0x3A, 0x38, 0x39, 0x00, 0x02]
    # relative error of a normal value is at most half a mantissa step, 2^-4
    x = np.random.default_rng(0).uniform(2.0 ** -6, 448.0, size=2000)
    assert np.max(np.abs(tab[enc(x)] - x) / x) <= 2.0 ** -4


def test_fp8_key_quantisation_exponent_and_exactness():
    # exponent = smallest e with max|k| 2^-e <= 448: 448 -> 0, 449 -> 1, 224 -> -1, 1 -> -8 (448/2^9 < 1 <= 448/2^8)
    K = np.zeros((5, 4))
    K[0] = [448.0, 1.0, 0.0, 0.0]; K[1] = [449.0, 0.0, 0.0, 0.0]; K[2] = [224.0, -3.0, 0.0, 0.0]
    K[3] = [1.0, 0.5, 0.0, 0.0]
    codes, exps, deq = so.quantize_keys_e4m3(K, 2)
    assert list(exps[:, 0]) == [0, 1, -1, -8, 0] and list(exps[:, 1]) == [0, 0, 0, 0, 0]
    assert deq[0, 0] == 448.0 and deq[1, 0] == 448.0 and deq[2, 0] == 224.0 and deq[3, 0] == 1.0 and deq[3, 1] == 0.5
    # values with at most 4 significant bits inside a head slice are stored exactly; others to 2^-4
    g = np.random.default_rng(1)
    K2 = synth.round_to_bf16(g.standard_normal((50, 64)) * g.uniform(0.01, 30.0, size=(50, 1))).astype(np.float64)
    c2, e2, d2 = so.quantize_keys_e4m3(K2, 4)
    amax = np.max(np.abs(K2.reshape(50, 4, 16)), axis=2)
    assert np.all(amax * np.exp2(-e2.astype(np.float64)) <= 448.0) and np.all(amax * np.exp2(-(e2 - 1.0)) > 448.0)
    err = np.abs(d2 - K2).reshape(50, 4, 16)
    assert np.all(err <= amax[:, :, None] * 2.0 ** -4)           # half a step of the largest binade at worst
    # the attention over the stored keys is ordinary slim attention on the dequantised rows
    W = g.standard_normal((64, 64)) / 8; q = g.standard_normal(64)
    assert np.array_equal(so.oracle_slim_fp8(q, K2, W, 4, 1.0e4), so.oracle_slim(q, d2, W, 4, 1.0e4))
    # and, for keys of ordinary size, close to the unquantised result (keys perturbed by <= 2^-4 of their slice maximum)
    K3 = synth.round_to_bf16(g.standard_normal((50, 64))).astype(np.float64)
    ref = so.oracle_slim(q, K3, W, 4, 1.0e4)
    assert so.err_rms_norm(so.oracle_slim_fp8(q, K3, W, 4, 1.0e4), ref) < 0.2


# ---- one context split into slices ---------------------------------------------------------------
def test_partials_of_any_split_join_to_the_whole_context():
    T, d, H = 77, 16, 2
    X, W_Q, W_K, W_V = _rand_case(50, T, d, H)
    K, q, W_KV = X @ W_K, X[-1] @ W_Q, so.oracle_wkv(W_K, W_V)
    for theta in (0.0, 1.0e4):
        whole = so.oracle_vanilla(X, W_Q, W_K, W_V, H, theta)
        for cuts in ([0, T], [0, 16, 48, T], [0, 32, 32, 64, T], [0, 1, T]):      # incl. an empty slice and a one-row slice
            parts = [so.oracle_slim_partial(q, K[a:b], a, T - 1, H, theta) for a, b in zip(cuts[:-1], cuts[1:])]
            out = so.oracle_combine_partials(np.stack([p[0] for p in parts]), np.stack([p[1] for p in parts]), W_KV)
            assert np.max(np.abs(out - whole)) <= 1e-10 * np.max(np.abs(whole))


def test_partial_hand_case_single_row_and_two_equal_rows():
    # one head of width 2, no RoPE.  One row k: lse = (q.k / sqrt 2) / ln 2, u = k.  Two identical rows: lse grows by exactly 1.
    q = np.array([2.0, 0.0]); k = np.array([[math.sqrt(2.0) * math.log(2.0) * 1.5, 7.0]])
    lse, u = so.oracle_slim_partial(q, k, 0, 0, 1, 0.0)
    assert abs(lse[0] - 3.0) < 1e-12 and np.array_equal(u[0], k[0])          # q.k / sqrt 2 = 3 ln 2
    lse2, u2 = so.oracle_slim_partial(q, np.vstack([k, k]), 0, 1, 1, 0.0)
    assert abs(lse2[0] - 4.0) < 1e-12 and np.allclose(u2[0], k[0])
    lse0, u0 = so.oracle_slim_partial(q, np.zeros((0, 2)), 0, 0, 1, 0.0)
    assert lse0[0] == -np.inf and np.all(u0 == 0)
    # join by hand: slices with lse 3 and 4 weigh 1/3 and 2/3
    out = so.oracle_combine_partials(np.array([[3.0], [4.0]]), np.array([[[3.0, 0.0]], [[0.0, 3.0]]]), np.eye(2))
    assert np.allclose(out, [1.0, 2.0])
