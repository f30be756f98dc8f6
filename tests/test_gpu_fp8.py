"""8-bit K-cache (one byte per cached value, the byte accounting of the paper's introduction) through the
C ABI: the library quantises appended bf16 rows to E4M3 codes with one power-of-two exponent per (row,
head); the oracle does the same from the published format.  Codes and exponents must agree bit for bit;
the attention over the stored keys must match the oracle within the bf16 tolerance (W_KV stays bf16)."""
import numpy as np
import pytest
import torch

from oracle import slim_oracle as so
from paper_2503_05840_b200 import binding as B
from paper_2503_05840_b200 import synth
from paper_2503_05840_b200.layer import SlimLayer, to_device_keys

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _stored(layer, batch, t_cap, d, H):
    raw = layer.k.cpu().numpy()
    n = batch * t_cap * d
    off = (n + 15) // 16 * 16
    return raw[:n].reshape(batch, t_cap, d), raw[off:off + batch * t_cap * H].view(np.int8).reshape(batch, t_cap, H)


@pytest.mark.parametrize("d,H,d_k,theta", [(512, 4, 128, 1.0e6), (1280, 20, 64, 0.0), (384, 4, 96, 1.0e4), (512, 32, 16, 1.0e4)])
def test_fp8_cache_codes_bitwise_and_decode_matches_oracle(d, H, d_k, theta):
    lengths = np.array([333, 0, 640, 17, 16, 1, 257], dtype=np.int32)
    batch, t_cap = len(lengths), 640
    cfg = synth.SlimConfig("fp8", d, H, d_k, batch, t_cap, 1, theta, "bf16")
    L = synth.make_layer(cfg, 61, lengths=lengths)
    K = L.K.copy()
    K[2, :200] *= np.exp2(np.random.default_rng(3).integers(-12, 12, size=(200, 1))).astype(np.float32)   # rows of very different size
    K[2, 5] = 0.0                                                                                    # an all-zero row
    K = synth.round_to_bf16(K)
    W_KV = so.oracle_wkv(L.W_K, L.W_V)
    layer = SlimLayer(d, H, d_k, theta, "fp8", batch, t_cap, DEV)
    try:
        assert B.slim_cache_bytes(layer.ctx, batch, t_cap) == (batch * t_cap * d + 15) // 16 * 16 + batch * t_cap * H
        layer.set_wkv(W_KV)
        Kd = to_device_keys(K, "bf16", DEV)
        q = to_device_keys(L.q, "bf16", DEV)
        ld = torch.from_numpy(lengths).to(DEV)
        # the prompt in bulk (all but the last row), then the newest row together with the decode
        bulk = int(lengths.max()) - 1
        layer.append_k(Kd[:, :bulk].contiguous(), torch.zeros(batch, dtype=torch.int32, device=DEV))
        k_new = torch.zeros((batch, d), dtype=torch.bfloat16, device=DEV)
        for b in range(batch):
            if lengths[b] > 0:
                k_new[b] = Kd[b, lengths[b] - 1]
        got = layer.decode_step(q, k_new, ld).cpu().numpy().astype(np.float64)
        assert layer.device_status() == B.SLIM_OK
        # shapes the tensor-core kernels take are decoded into a bf16 scratch and run there; the others stay on CUDA cores
        probe = B.slim_create(d, H, d_k, theta, B.SLIM_BF16)       # what a bf16 cache of this shape would run on
        B.slim_set_wkv(probe, np.eye(d))
        tc_shape = B.slim_query(probe, B.SLIM_Q_PATH_IN_USE) == B.SLIM_PATH_TC
        B.slim_destroy(probe)
        assert layer.query(B.SLIM_Q_PATH_IN_USE) == (B.SLIM_PATH_TC if tc_shape else B.SLIM_PATH_GENERIC)
        codes, exps = _stored(layer, batch, t_cap, d, H)
        for b in range(batch):
            n = int(lengths[b])
            if n == 0:
                assert np.all(got[b] == 0)
                continue
            c_ref, e_ref, deq = so.quantize_keys_e4m3(K[b, :n], H)
            assert np.array_equal(codes[b, :n], c_ref), f"sequence {b}: codes differ"
            assert np.array_equal(exps[b, :n], e_ref), f"sequence {b}: exponents differ"
            ref = so.oracle_slim(L.q[b], deq, W_KV, H, theta)
            e = so.err_rms_norm(got[b], ref)
            assert e <= 2e-2, f"sequence {b}: {e:.3e}"
        # plain decode over the stored keys gives the same bits as the step call did
        again = layer.decode(q, ld).cpu().numpy().astype(np.float64)
        assert np.array_equal(again, got)
        if tc_shape:
            # the CUDA-core kernels read the same codes directly: same tolerance against the oracle
            layer.set_path(B.SLIM_PATH_GENERIC)
            gen = layer.decode(q, ld).cpu().numpy().astype(np.float64)
            assert layer.device_status() == B.SLIM_OK
            for b in range(batch):
                n = int(lengths[b])
                if n == 0:
                    assert np.all(gen[b] == 0)
                    continue
                _, _, deq = so.quantize_keys_e4m3(K[b, :n], H)
                e = so.err_rms_norm(gen[b], so.oracle_slim(L.q[b], deq, W_KV, H, theta))
                assert e <= 2e-2, f"CUDA-core path, sequence {b}: {e:.3e}"
    finally:
        layer.close()


def test_fp8_cache_refuses_what_it_does_not_support():
    ctx = B.slim_create(256, 16, 16, 0.0, B.SLIM_FP8)          # (d_k = 16: no tensor-core kernel for this shape)
    try:
        with pytest.raises(B.SlimError) as ei:
            B.slim_xcache_set_weights(ctx, np.eye(256), np.eye(256))
        assert ei.value.status == B.SLIM_ERR_UNSUPPORTED
        pool = torch.zeros(64 * 32 * 256, dtype=torch.uint8, device=DEV)
        table = torch.zeros((2, 4), dtype=torch.int32, device=DEV)
        with pytest.raises(B.SlimError) as ei:
            B.slim_cache_create_paged(ctx, pool, 8, 32, table, 2, 4)
        assert ei.value.status == B.SLIM_ERR_UNSUPPORTED
        with pytest.raises(B.SlimError):
            B.slim_set_path(ctx, B.SLIM_PATH_TC)
    finally:
        B.slim_destroy(ctx)
