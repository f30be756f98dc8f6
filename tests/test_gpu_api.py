"""GPU tests of the boundary: set_weights against the oracle, append, error
statuses, and properties that hold at any size."""
import numpy as np
import pytest
import torch

from oracle import slim_oracle as so
from paper_2503_05840_b200 import binding as B
from paper_2503_05840_b200 import synth
from paper_2503_05840_b200.layer import SlimLayer, to_device_keys

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.mark.parametrize("d,H", [(32, 2), (96, 3), (384, 6), (1000, 10), (1280, 20)])
def test_set_weights_matches_oracle_and_closed_form(d, H):
    W_Q, W_K, W_V, Qo, s = synth.make_weights(d, 77 + d)
    layer = SlimLayer(d, H, d // H, 0.0, "f32", 1, 16, DEV)
    try:
        res, wkv = layer.set_weights(W_K, W_V, want_wkv=True)
        ref = so.oracle_wkv(W_K, W_V)
        closed = (Qo.T @ W_V) / s[:, None]
        assert np.allclose(wkv, ref, rtol=1e-9, atol=1e-11)
        assert np.allclose(wkv, closed, rtol=1e-9, atol=1e-11)
        assert res <= 1e-12 * d
        assert np.allclose(W_K @ wkv, W_V)          # the appendix-A check
        # float32 host weights are accepted too
        res32, wkv32 = layer.set_weights(W_K.astype(np.float32), W_V.astype(np.float32), want_wkv=True)
        ref32 = so.oracle_wkv(W_K.astype(np.float32).astype(np.float64), W_V.astype(np.float32).astype(np.float64))
        assert np.allclose(wkv32, ref32, rtol=1e-8, atol=1e-10)
    finally:
        layer.close()


def test_set_weights_general_matrix_with_pivoting():
    g = np.random.default_rng(5)
    d = 192
    W_K = g.standard_normal((d, d))
    W_K[0, 0] = 0.0                       # forces a row exchange at the first step
    W_V = g.standard_normal((d, d))
    layer = SlimLayer(d, 4, d // 4, 0.0, "f32", 1, 16, DEV)
    try:
        res, wkv = layer.set_weights(W_K, W_V, want_wkv=True)
        ref = so.oracle_wkv(W_K, W_V)
        assert np.max(np.abs(wkv - ref)) <= 1e-8 * np.max(np.abs(ref))
    finally:
        layer.close()


def test_singular_w_k_is_reported():
    d = 64
    W_K = np.ones((d, d))
    layer = SlimLayer(d, 2, 32, 0.0, "f32", 1, 16, DEV)
    try:
        with pytest.raises(B.SlimError) as ei:
            layer.set_weights(W_K, np.eye(d))
        assert ei.value.status == B.SLIM_ERR_SINGULAR
        q = torch.zeros((1, d), device=DEV)
        with pytest.raises(B.SlimError) as ei:
            layer.decode(q, torch.ones(1, dtype=torch.int32, device=DEV))
        assert ei.value.status == B.SLIM_ERR_NO_WEIGHTS
    finally:
        layer.close()


def test_set_wkv_equals_set_weights():
    cfg = synth.SlimConfig("x", 256, 4, 64, 2, 64, 1, 1.0e4, "bf16")
    L = synth.make_layer(cfg, 31)
    outs = []
    for mode in ("solve", "direct"):
        layer = SlimLayer(cfg.d, cfg.H, cfg.d_k, cfg.rope_theta, cfg.dtype, cfg.batch, cfg.context, DEV)
        try:
            layer.k.copy_(to_device_keys(L.K, cfg.dtype, DEV))
            if mode == "solve":
                layer.set_weights(L.W_K, L.W_V)
            else:
                layer.set_wkv(so.oracle_wkv(L.W_K, L.W_V))
            q = to_device_keys(L.q, cfg.dtype, DEV)
            outs.append(layer.decode(q, torch.from_numpy(L.lengths).to(DEV)).cpu().numpy())
        finally:
            layer.close()
    assert np.allclose(outs[0], outs[1], rtol=1e-5, atol=1e-6)


@pytest.mark.parametrize("dtype,theta", [("f32", 0.0), ("bf16", 1.0e4)])
def test_append_then_decode_equals_prefilled_cache(dtype, theta):
    cfg = synth.SlimConfig("app", 256, 4, 64, 3, 80, 1, theta, dtype)
    lengths = np.array([80, 37, 5], dtype=np.int32)
    L = synth.make_layer(cfg, 555, lengths=lengths)
    W_KV = so.oracle_wkv(L.W_K, L.W_V)
    a = SlimLayer(cfg.d, cfg.H, cfg.d_k, theta, dtype, cfg.batch, cfg.context, DEV)
    b = SlimLayer(cfg.d, cfg.H, cfg.d_k, theta, dtype, cfg.batch, cfg.context, DEV)
    try:
        Kd = to_device_keys(L.K, dtype, DEV)
        a.k.copy_(Kd)
        a.set_wkv(W_KV); b.set_wkv(W_KV)
        # b: feed the keys through slim_append_k, first a bulk of len-3 rows, then three single rows
        pos = torch.zeros(3, dtype=torch.int32, device=DEV)
        bulk = int(lengths.min()) - 3
        b.append_k(Kd[:, :bulk].contiguous(), pos)
        cur = np.full(3, bulk, dtype=np.int32)
        while np.any(cur < lengths):
            step = torch.zeros((3, 1, cfg.d), dtype=Kd.dtype, device=DEV)
            posd = torch.from_numpy(np.minimum(cur, lengths - 1).astype(np.int32)).to(DEV)
            for i in range(3):
                step[i, 0] = Kd[i, min(cur[i], lengths[i] - 1)]
            b.append_k(step, posd)
            cur = np.minimum(cur + 1, lengths)
        assert b.device_status() == B.SLIM_OK
        for i in range(3):
            assert torch.equal(b.k[i, :lengths[i]], a.k[i, :lengths[i]])
        q = to_device_keys(L.q, dtype, DEV)
        ld = torch.from_numpy(lengths).to(DEV)
        oa = a.decode(q, ld).clone()
        ob = b.decode(q, ld).clone()
        assert torch.equal(oa, ob)
    finally:
        a.close(); b.close()


def test_append_beyond_capacity_sets_status_and_writes_nothing():
    layer = SlimLayer(64, 2, 32, 0.0, "f32", 2, 8, DEV)
    try:
        layer.k.fill_(7.0)
        k_new = torch.ones((2, 2, 64), device=DEV)
        layer.append_k(k_new, torch.tensor([7, 0], dtype=torch.int32, device=DEV))   # seq 0: rows 7,8 -> overflow
        assert layer.device_status() == B.SLIM_ERR_CAPACITY
        assert layer.device_status() == B.SLIM_OK            # status is cleared by the read
        assert torch.all(layer.k[0] == 7.0)
        assert torch.all(layer.k[1, :2] == 1.0) and torch.all(layer.k[1, 2:] == 7.0)
    finally:
        layer.close()


def test_append_at_a_huge_position_is_refused_not_wrapped():
    """A garbage position near INT_MAX must not wrap around the capacity check (the comparison is made
    without adding to the position): status CAPACITY, no row written."""
    layer = SlimLayer(64, 2, 32, 0.0, "f32", 2, 8, DEV)
    try:
        layer.k.fill_(7.0)
        k_new = torch.ones((2, 2, 64), device=DEV)
        layer.append_k(k_new, torch.tensor([2**31 - 1, 2**31 - 2], dtype=torch.int32, device=DEV))
        assert layer.device_status() == B.SLIM_ERR_CAPACITY
        assert torch.all(layer.k == 7.0)
    finally:
        layer.close()


def test_length_beyond_capacity_is_clamped_and_reported():
    cfg = synth.SlimConfig("cap", 128, 2, 64, 1, 40, 1, 0.0, "f32")
    L = synth.make_layer(cfg, 3)
    layer = SlimLayer(cfg.d, cfg.H, cfg.d_k, 0.0, "f32", 1, 40, DEV)
    try:
        layer.k.copy_(to_device_keys(L.K, "f32", DEV))
        layer.set_weights(L.W_K, L.W_V)
        q = to_device_keys(L.q, "f32", DEV)
        good = layer.decode(q, torch.tensor([40], dtype=torch.int32, device=DEV)).clone()
        assert layer.device_status() == B.SLIM_OK
        got = layer.decode(q, torch.tensor([41], dtype=torch.int32, device=DEV)).clone()
        assert layer.device_status() == B.SLIM_ERR_CAPACITY
        assert torch.equal(got, good)
    finally:
        layer.close()


def _paths(layer):
    paths = [B.SLIM_PATH_GENERIC]
    try:
        layer.set_path(B.SLIM_PATH_TC); paths.append(B.SLIM_PATH_TC)
    except B.SlimError:
        pass
    layer.set_path(B.SLIM_PATH_AUTO)
    return paths


def test_poisoned_rows_beyond_length_do_not_leak_and_runs_are_bitwise_repeatable():
    cfg = synth.SlimConfig("poison", 1024, 8, 128, 4, 700, 1, 1.0e6, "bf16")
    lengths = np.array([700, 333, 17, 640], dtype=np.int32)
    L = synth.make_layer(cfg, 42, lengths=lengths)
    layer = SlimLayer(cfg.d, cfg.H, cfg.d_k, cfg.rope_theta, "bf16", cfg.batch, cfg.context, DEV)
    try:
        Kd = to_device_keys(L.K, "bf16", DEV)
        layer.set_weights(L.W_K, L.W_V)
        q = to_device_keys(L.q, "bf16", DEV)
        ld = torch.from_numpy(lengths).to(DEV)
        for path in _paths(layer):
            layer.set_path(path)
            layer.k.copy_(Kd)
            clean = layer.decode(q, ld).clone()
            for b in range(4):
                layer.k[b, lengths[b]:] = float("nan")
            nan_run = layer.decode(q, ld).clone()
            for b in range(4):
                layer.k[b, lengths[b]:] = float("inf")
            inf_run = layer.decode(q, ld).clone()
            assert torch.equal(clean, nan_run), f"path {path}"
            assert torch.equal(clean, inf_run), f"path {path}"
            again = layer.decode(q, ld).clone()
            assert torch.equal(inf_run, again)
    finally:
        layer.close()


def test_row_permutation_invariance_without_rope_and_identical_keys():
    cfg = synth.SlimConfig("perm", 1280, 20, 64, 2, 1500, 1, 0.0, "bf16")
    L = synth.make_layer(cfg, 8)
    layer = SlimLayer(cfg.d, cfg.H, cfg.d_k, 0.0, "bf16", cfg.batch, cfg.context, DEV)
    try:
        Kd = to_device_keys(L.K, "bf16", DEV)
        W_KV = so.oracle_wkv(L.W_K, L.W_V)
        layer.set_wkv(W_KV)
        q = to_device_keys(L.q, "bf16", DEV)
        ld = torch.from_numpy(L.lengths).to(DEV)
        g = torch.Generator(device="cpu"); g.manual_seed(0)
        perm = torch.randperm(1500, generator=g).to(DEV)
        for path in _paths(layer):
            layer.set_path(path)
            layer.k.copy_(Kd)
            base = layer.decode(q, ld).clone()
            layer.k.copy_(Kd[:, perm])
            shuffled = layer.decode(q, ld).clone()
            # The order of the rows changes the softmax reference exponent and with it
            # the bf16 rounding of every probability (relative 2^-9 each), so the two
            # runs differ by rounding noise, not bit for bit: half the parity bound.
            rms = base.pow(2).mean().sqrt()
            assert (base - shuffled).abs().max() <= 1e-2 * rms
            # all keys identical: the output is that key's value row, whatever q is
            layer.k.copy_(Kd[:, :1].expand(-1, 1500, -1))
            same = layer.decode(q, ld).cpu().numpy().astype(np.float64)
            for b in range(2):
                v = L.K[b, 0].astype(np.float64) @ W_KV
                assert so.err_rms_norm(same[b], v) <= 2e-2
    finally:
        layer.close()


@pytest.mark.parametrize("d,H,d_k", [(512, 4, 128), (256, 4, 64)])
def test_scores_far_above_the_first_tile_are_handled(d, H, d_k):
    # later keys score much higher than the first tile's: exercises the
    # reference-exponent handling of every path (and its exact redo, if any);
    # d_k = 64 runs the kernel with two score-warp sets, either of which may raise the flag.
    cfg = synth.SlimConfig("ramp", d, H, d_k, 2, 400, 1, 0.0, "bf16")
    L = synth.make_layer(cfg, 77)
    K = L.K.copy()
    q = L.q.copy()
    for b in range(2):
        qn = q[b] / np.linalg.norm(q[b])
        ramp = np.linspace(0.0, 60.0 if b == 0 else 400.0, 400)[:, None]
        K[b] = synth.round_to_bf16(K[b] + ramp * qn[None, :] * 8.0)
    layer = SlimLayer(cfg.d, cfg.H, cfg.d_k, 0.0, "bf16", cfg.batch, cfg.context, DEV)
    try:
        W_KV = so.oracle_wkv(L.W_K, L.W_V)
        layer.set_wkv(W_KV)
        layer.k.copy_(to_device_keys(K, "bf16", DEV))
        qd = to_device_keys(q, "bf16", DEV)
        ld = torch.from_numpy(L.lengths).to(DEV)
        ref = so.oracle_slim_batch(q, K, L.lengths, W_KV, cfg.H, 0.0)
        for path in _paths(layer):
            layer.set_path(path)
            got = layer.decode(qd, ld).cpu().numpy().astype(np.float64)
            assert layer.device_status() == B.SLIM_OK
            for b in range(2):
                assert so.err_rms_norm(got[b], ref[b]) <= 2e-2, f"path {path} seq {b}"
    finally:
        layer.close()


def test_bounded_wait_gives_up_reports_timeout_and_context_survives():
    # a wait that nothing completes must run out, not hang: status TIMEOUT, then normal work again
    cfg = synth.SlimConfig("wait", 256, 2, 128, 2, 64, 1, 1.0e4, "bf16")
    L = synth.make_layer(cfg, 5)
    layer = SlimLayer(cfg.d, cfg.H, cfg.d_k, cfg.rope_theta, "bf16", cfg.batch, cfg.context, DEV)
    try:
        layer.k.copy_(to_device_keys(L.K, "bf16", DEV))
        W_KV = so.oracle_wkv(L.W_K, L.W_V)
        layer.set_wkv(W_KV)
        q = to_device_keys(L.q, "bf16", DEV)
        ld = torch.from_numpy(L.lengths).to(DEV)
        before = layer.decode(q, ld).clone()
        assert layer.device_status() == B.SLIM_OK
        B.slim_selftest_bounded_wait(layer.ctx, torch.cuda.current_stream().cuda_stream)
        assert layer.device_status() == B.SLIM_ERR_TIMEOUT
        assert layer.device_status() == B.SLIM_OK
        after = layer.decode(q, ld).clone()
        assert layer.device_status() == B.SLIM_OK
        assert torch.equal(before, after)
    finally:
        layer.close()


def test_nonsquare_weights_right_inverse_matches_oracle_and_decodes():
    # d_model = 192 < e = H d_k = 512: W_KV is e x e (non-square section, Option 1)
    d_model, e, H, d_k, T = 192, 512, 4, 128, 300
    W_Q, W_K, W_V, Qrows, s = synth.make_weights_nonsquare(d_model, e, 21)
    g = np.random.default_rng(2)
    lengths = np.array([T, 77], dtype=np.int32)
    layer = SlimLayer(e, H, d_k, 1.0e4, "bf16", 2, T, DEV)
    try:
        with torch.cuda.device(DEV):
            res, wkv = B.slim_set_weights_nonsquare(layer.ctx, W_K, W_V, want_wkv=True)
        ref = so.oracle_wkv_right_inverse(W_K, W_V)
        assert np.allclose(wkv, ref, rtol=1e-8, atol=1e-10)
        assert np.allclose(wkv, Qrows.T @ (W_V / s[:, None]), rtol=1e-8, atol=1e-10)
        assert res < 1e-10
        K = np.zeros((2, T, e), dtype=np.float32); q = np.zeros((2, e), dtype=np.float32)
        Xs = []
        for b in range(2):
            X = g.standard_normal((int(lengths[b]), d_model)); Xs.append(X)
            K[b, :lengths[b]] = synth.round_to_bf16(X @ W_K); q[b] = synth.round_to_bf16(X[-1] @ W_Q)
        layer.k.copy_(to_device_keys(K, "bf16", DEV))
        got = layer.decode(to_device_keys(q, "bf16", DEV), torch.from_numpy(lengths).to(DEV)).cpu().numpy().astype(np.float64)
        assert layer.device_status() == B.SLIM_OK
        for b in range(2):
            slim = so.oracle_slim(q[b], K[b, :lengths[b]], ref, H, 1.0e4)
            assert so.err_rms_norm(got[b], slim) <= 2e-2
            # and, up to the bf16 rounding of K and q, the vanilla result with an explicit V = X W_V
            van = so.oracle_vanilla(Xs[b], W_Q, W_K, W_V, H, 1.0e4)
            assert so.err_rms_norm(got[b], van) <= 5e-2
        # a rank-deficient W_K has no right inverse
        bad = W_K.copy(); bad[1] = bad[0]
        with pytest.raises(B.SlimError) as ei:
            with torch.cuda.device(DEV):
                B.slim_set_weights_nonsquare(layer.ctx, bad, W_V)
        assert ei.value.status == B.SLIM_ERR_SINGULAR
    finally:
        layer.close()


@pytest.mark.parametrize("d,H,d_k,dtype", [(512, 4, 128, "bf16"), (1280, 20, 64, "bf16"), (384, 4, 96, "bf16"), (256, 4, 64, "f32"), (192, 2, 96, "bf16"),
                                          (384, 6, 64, "bf16"), (384, 3, 128, "bf16")])
def test_prompt_phase_values_from_keys(d, H, d_k, dtype):
    # Fig. 3(a): V = K W_KV for a whole prompt; equals X W_V up to the rounding of the stored keys
    n = 300
    W_Q, W_K, W_V, _, _ = synth.make_weights(d, 300 + d)
    X = np.random.default_rng(d).standard_normal((n, d))
    K = synth.round_to_dtype(X @ W_K, dtype)
    layer = SlimLayer(d, H, d_k, 0.0, dtype, 1, 16, DEV)
    try:
        layer.set_weights(W_K, W_V)
        Kd = to_device_keys(K, dtype, DEV)
        V = torch.full((n, d), float("nan"), dtype=torch.float32, device=DEV)
        with torch.cuda.device(DEV):
            B.slim_values_from_keys(layer.ctx, Kd, n, V, torch.cuda.current_stream().cuda_stream)
        assert layer.device_status() == B.SLIM_OK
        got = V.cpu().numpy().astype(np.float64)
        assert np.all(np.isfinite(got))
        ref = K.astype(np.float64) @ so.oracle_wkv(W_K, W_V)          # Eq. 6 on the stored keys
        van = X @ W_V                                                  # Eq. 5
        tol = 2e-2 if dtype == "bf16" else 1e-4
        for t in (0, 1, 127, 128, 255, 299):
            e = so.err_rms_norm(got[t], ref[t]) if dtype == "bf16" else so.err_fp32_norm(got[t], ref[t])
            assert e <= tol, f"row {t}: {e:.3e}"
            assert so.err_rms_norm(got[t], van[t]) <= (5e-2 if dtype == "bf16" else 1e-3)
        worst = max(so.err_rms_norm(got[t], ref[t]) for t in range(n))
        assert worst <= (2e-2 if dtype == "bf16" else 1e-4)
    finally:
        layer.close()


@pytest.mark.parametrize("d,H,d_k,theta,dtype", [(512, 4, 128, 1.0e6, "bf16"), (1280, 20, 64, 0.0, "bf16"),
                                                 (384, 4, 96, 1.0e4, "bf16"), (384, 6, 64, 0.0, "f32")])
def test_decode_step_equals_append_then_decode(d, H, d_k, theta, dtype):
    """slim_decode_step (cache update + attention in one call) against slim_append_k + slim_decode on a
    second, identical cache: same output bits, same cache bits afterwards; sequence lengths at tile
    edges, an empty sequence (nothing written) and the oracle on top."""
    lengths = np.array([333, 0, 640, 17, 16, 1, 257], dtype=np.int32)      # lengths AFTER the update
    batch, t_cap = len(lengths), 640
    cfg = synth.SlimConfig("step", d, H, d_k, batch, t_cap, 1, theta, dtype)
    L = synth.make_layer(cfg, 31, lengths=lengths)
    W_KV = so.oracle_wkv(L.W_K, L.W_V)
    a = SlimLayer(d, H, d_k, theta, dtype, batch, t_cap, DEV)
    b_ = SlimLayer(d, H, d_k, theta, dtype, batch, t_cap, DEV)
    try:
        Kd = to_device_keys(L.K, dtype, DEV)
        k_new = torch.zeros((batch, d), dtype=Kd.dtype, device=DEV)
        before = Kd.clone()
        for b in range(batch):
            if lengths[b] > 0:
                k_new[b] = Kd[b, lengths[b] - 1]
                before[b, lengths[b] - 1] = 123.0              # the row the step has to overwrite
            before[b, lengths[b]:] = float("nan")              # rows past the end are poison
        k_new[1] = 55.0                                        # empty sequence: must not be written anywhere
        q = to_device_keys(L.q, dtype, DEV)
        ld = torch.from_numpy(lengths).to(DEV)
        ref = so.oracle_slim_batch(L.q, L.K, lengths, W_KV, H, theta)
        tol = 2e-2 if dtype == "bf16" else 1e-4
        for path in _paths(a):
            for lay in (a, b_):
                lay.set_path(path); lay.set_wkv(W_KV); lay.k.copy_(before)
            got = a.decode_step(q, k_new, ld).clone()
            assert a.device_status() == B.SLIM_OK
            b_.append_k(k_new.unsqueeze(1).contiguous(), (ld - 1).clamp(min=0))
            # (the append call writes row 0 of the empty sequence; the step call must not)
            want = b_.decode(q, ld).clone()
            assert torch.equal(got, want), f"path {path}"
            ka, kb = a.k.clone(), b_.k.clone()
            assert torch.equal(ka[1].isnan(), before[1].isnan()) and not (ka[1] == 55.0).any()
            kb[1] = ka[1]
            assert torch.equal(torch.nan_to_num(ka, nan=-7.0), torch.nan_to_num(kb, nan=-7.0)), f"path {path}: cache differs"
            g = got.cpu().numpy().astype(np.float64)
            for b in range(batch):
                if lengths[b] == 0:
                    assert np.all(g[b] == 0)
                else:
                    e = so.err_rms_norm(g[b], ref[b]) if dtype == "bf16" else so.err_fp32_norm(g[b], ref[b])
                    assert e <= tol, f"path {path} seq {b}: {e:.3e}"
    finally:
        a.close(); b_.close()


def test_decode_step_capacity_and_launch_count():
    cfg = synth.SlimConfig("stepcap", 512, 4, 128, 2, 64, 1, 1.0e4, "bf16")
    L = synth.make_layer(cfg, 5)
    layer = SlimLayer(cfg.d, cfg.H, cfg.d_k, cfg.rope_theta, "bf16", 2, 64, DEV)
    try:
        layer.set_wkv(so.oracle_wkv(L.W_K, L.W_V))
        layer.k.copy_(to_device_keys(L.K, "bf16", DEV))
        q = to_device_keys(L.q, "bf16", DEV)
        k_new = torch.full((2, 512), 9.0, dtype=torch.bfloat16, device=DEV)
        keep = layer.k.clone()
        layer.decode_step(q, k_new, torch.tensor([65, 64], dtype=torch.int32, device=DEV))
        assert layer.device_status() == B.SLIM_ERR_CAPACITY          # sequence 0: beyond t_cap, nothing written
        assert torch.equal(layer.k[0], keep[0])
        assert torch.all(layer.k[1, 63] == 9.0) and torch.equal(layer.k[1, :63], keep[1, :63])
        # tensor-core path: decode kernel, column-split combine (so small a batch), projection (which makes its own
        # operand tiles from the combined rows); the update needs no kernel of its own
        assert layer.query(B.SLIM_Q_PATH_IN_USE) == B.SLIM_PATH_TC
        assert layer.query(B.SLIM_Q_LAUNCHES_PER_DECODE) == 3
        layer.set_path(B.SLIM_PATH_GENERIC)
        layer.decode_step(q, k_new, torch.tensor([3, 64], dtype=torch.int32, device=DEV))
        assert layer.device_status() == B.SLIM_OK
        assert layer.query(B.SLIM_Q_LAUNCHES_PER_DECODE) == 5         # append, scores, accumulation, column-split combine, projection
    finally:
        layer.close()


def test_scores_far_above_the_first_tile_with_rope_and_long_units():
    """Keys whose size grows along the context, with RoPE: arguments run hundreds of units above the
    first tile's in several heads and units, so whole sequences take the exact recomputation inside
    the combine kernel (rotation included); a third sequence stays ordinary."""
    d, H, d_k, theta = 512, 4, 128, 1.0e4
    lengths = np.array([3000, 1500, 900], dtype=np.int32)
    cfg = synth.SlimConfig("ramp-rope", d, H, d_k, 3, 3000, 1, theta, "bf16")
    L = synth.make_layer(cfg, 78, lengths=lengths)
    K = L.K.copy()
    for b in range(2):
        n = int(lengths[b])
        K[b, :n] = synth.round_to_bf16(K[b, :n] * (1.0 + np.arange(n)[:, None] * (0.5 if b == 0 else 0.05)))
    layer = SlimLayer(d, H, d_k, theta, "bf16", 3, 3000, DEV)
    try:
        W_KV = so.oracle_wkv(L.W_K, L.W_V)
        layer.set_wkv(W_KV)
        layer.k.copy_(to_device_keys(K, "bf16", DEV))
        qd = to_device_keys(L.q, "bf16", DEV)
        ld = torch.from_numpy(lengths).to(DEV)
        ref = so.oracle_slim_batch(L.q, K, lengths, W_KV, H, theta)
        for path in _paths(layer):
            layer.set_path(path)
            got = layer.decode(qd, ld).cpu().numpy().astype(np.float64)
            assert layer.device_status() == B.SLIM_OK
            for b in range(3):
                assert so.err_rms_norm(got[b], ref[b]) <= 2e-2, f"path {path} seq {b}"
    finally:
        layer.close()


@pytest.mark.parametrize("d,H,d_k,dtype,paged", [(512, 4, 128, "bf16", False), (1280, 20, 64, "bf16", False),
                                                 (512, 4, 128, "bf16", True), (256, 4, 64, "f32", False)])
def test_prefill_stores_the_keys_and_returns_their_values(d, H, d_k, dtype, paged):
    """slim_prefill (Fig. 3(a) in one call): several 128-row tiles with a ragged last one, three
    sequences, rows landing at different first positions; V against the oracle on every row, the
    cache bit for bit against the keys, rows outside the prompt untouched, a sequence without room
    refused."""
    batch, n_new, t_cap = 3, 293, 640
    g = np.random.default_rng(d + n_new)
    W_Q, W_K, W_V, _, _ = synth.make_weights(d, 400 + d)
    X = g.standard_normal((batch, n_new, d))
    K = synth.round_to_dtype(X @ W_K, dtype)
    W_KV = so.oracle_wkv(W_K, W_V)
    layer = SlimLayer(d, H, d_k, 0.0, dtype, batch, t_cap, DEV)
    try:
        layer.set_weights(W_K, W_V)
        Kd = to_device_keys(K, dtype, DEV)
        pos = np.array([0, 100, 347], dtype=np.int32)
        st = torch.cuda.current_stream().cuda_stream
        cache, table = layer.cache, None
        if paged:
            pr = 32
            mp = t_cap // pr
            perm = g.permutation(batch * mp).astype(np.int32).reshape(batch, mp)
            table = torch.from_numpy(perm).to(DEV)
            cache = B.slim_cache_create_paged(layer.ctx, layer.k, batch * mp, pr, table, batch, mp)
        layer.k.fill_(-3.0)
        V = torch.full((batch, n_new, d), float("nan"), dtype=torch.float32, device=DEV)
        with torch.cuda.device(DEV):
            B.slim_prefill(layer.ctx, cache, Kd, torch.from_numpy(pos).to(DEV), n_new, V, st)
        assert layer.device_status() == B.SLIM_OK
        got = V.cpu().numpy().astype(np.float64)
        tol = 2e-2 if dtype == "bf16" else 1e-4
        for b in range(batch):
            ref = so.oracle_prompt_values(K[b], W_KV)
            worst = max((so.err_rms_norm(got[b, t], ref[t]) if dtype == "bf16" else so.err_fp32_norm(got[b, t], ref[t]))
                        for t in range(n_new))
            assert worst <= tol, f"sequence {b}: {worst:.3e}"
        stored = layer.k.clone()
        if paged:
            rows = stored.reshape(batch * mp, pr, d)[table.long()].reshape(batch, t_cap, d)
        else:
            rows = stored
        for b in range(batch):
            assert torch.equal(rows[b, pos[b]:pos[b] + n_new], Kd[b]), f"sequence {b}: cache differs from the keys"
            assert torch.all(rows[b, :pos[b]] == -3.0) and torch.all(rows[b, pos[b] + n_new:] == -3.0)
        # no room for sequence 2: refused, nothing of it written, the other two stored
        layer.k.fill_(-3.0)
        with torch.cuda.device(DEV):
            B.slim_prefill(layer.ctx, cache, Kd, torch.tensor([0, 0, 348], dtype=torch.int32, device=DEV), n_new, V, st)
        assert layer.device_status() == B.SLIM_ERR_CAPACITY
        stored = layer.k.clone()
        rows = stored.reshape(batch * mp, pr, d)[table.long()].reshape(batch, t_cap, d) if paged else stored
        assert torch.all(rows[2] == -3.0) and torch.equal(rows[1, :n_new], Kd[1])
        if paged:
            B.slim_cache_destroy(cache)
    finally:
        layer.close()
