"""slim_decode_static_ws: the decode entry point for callers that are not allowed to
allocate device memory (a serving loop with a frozen memory pool, a plug-in on a device
it does not own).  Its scratch is a fixed array inside the library, so the test checks
that it gives the same output as slim_decode with a caller-owned workspace (and the oracle's,
within the usual tolerance) -- twice in a row, because the second call starts from whatever
the first left in the shared array, and after a call of another shape has left its own
scratch there -- that the free device memory is the same before and after the calls, and
that a shape whose scratch need is above the built-in maximum is refused before anything
is launched.  Collected last on purpose (file name)."""
import numpy as np
import pytest
import torch

from oracle import slim_oracle as so
from paper_2503_05840_b200 import binding as B
from paper_2503_05840_b200 import synth
from paper_2503_05840_b200.layer import SlimLayer, to_device_keys

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _dirty_the_static_scratch():
    """A call of another shape (fp32, CUDA-core kernels, other unit count) leaves its partials, flags
    and slices in the shared array."""
    cfg = synth.SlimConfig("dirty", 256, 4, 64, 5, 90, 1, 0.0, "f32")
    L = synth.make_layer(cfg, 777, lengths=np.array([90, 1, 33, 64, 7], dtype=np.int32))
    layer = SlimLayer(256, 4, 64, 0.0, "f32", 5, 90, DEV)
    try:
        layer.k.copy_(to_device_keys(L.K, "f32", DEV))
        layer.set_weights(L.W_K, L.W_V)
        o = torch.empty((5, 256), dtype=torch.float32, device=DEV)
        with torch.cuda.device(DEV):
            B.slim_decode_static_ws(layer.ctx, to_device_keys(L.q, "f32", DEV), layer.cache,
                                    torch.from_numpy(L.lengths).to(DEV), o, torch.cuda.current_stream().cuda_stream)
        assert layer.device_status() == B.SLIM_OK
    finally:
        layer.close()


@pytest.mark.parametrize("d,H,d_k,theta,dtype,tol", [
    (512, 4, 128, 1.0e4, "bf16", 2e-2),     # tensor-core path
    (384, 6, 64, 0.0, "f32", 1e-4),         # CUDA-core path
])
def test_static_workspace_decode_matches_decode_twice(d, H, d_k, theta, dtype, tol):
    _dirty_the_static_scratch()
    lengths = np.array([600, 333, 17], dtype=np.int32)
    cfg = synth.SlimConfig("noalloc", d, H, d_k, 3, 600, 1, theta, dtype)
    L = synth.make_layer(cfg, 4242, lengths=lengths)
    layer = SlimLayer(d, H, d_k, theta, dtype, 3, 600, DEV)
    try:
        assert B.slim_workspace_bytes(layer.ctx, 3, 600) <= B.slim_static_workspace_max()
        layer.k.copy_(to_device_keys(L.K, dtype, DEV))
        layer.set_weights(L.W_K, L.W_V)
        q = to_device_keys(L.q, dtype, DEV)
        ld = torch.from_numpy(lengths).to(DEV)
        want = layer.decode(q, ld).clone()
        assert layer.device_status() == B.SLIM_OK
        stream = torch.cuda.current_stream().cuda_stream
        ref = so.oracle_slim_batch(L.q, L.K, lengths, so.oracle_wkv(L.W_K, L.W_V), H, theta)
        outs = [torch.full((3, d), float("nan"), dtype=torch.float32, device=DEV) for _ in range(2)]
        other = torch.empty_like(outs[0])
        q_flipped = torch.flip(q, dims=[0]).contiguous()
        # the three calls run with nothing else between them, so a change of the free device
        # memory could only come from the entry point itself
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        with torch.cuda.device(DEV):
            B.slim_decode_static_ws(layer.ctx, q, layer.cache, ld, outs[0], stream)
            # a different query in between, so the second call really recomputes over stale scratch
            B.slim_decode_static_ws(layer.ctx, q_flipped, layer.cache, ld, other, stream)
            B.slim_decode_static_ws(layer.ctx, q, layer.cache, ld, outs[1], stream)
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free_before, "device memory in use changed across the calls"
        assert layer.device_status() == B.SLIM_OK
        for call, o in enumerate(outs):
            assert torch.isfinite(o).all(), f"call {call}"
            rms = want.pow(2).mean(dim=1, keepdim=True).sqrt()
            if dtype == "bf16":
                err = ((o - want).abs() / rms).max().item()
            else:
                err = ((o - want).abs() / torch.maximum(want.abs(), rms)).max().item()
            assert err <= tol, f"call {call}: {err:.3e}"
            got = o.cpu().numpy().astype(np.float64)
            for b in range(3):
                e = so.err_rms_norm(got[b], ref[b]) if dtype == "bf16" else so.err_fp32_norm(got[b], ref[b])
                assert e <= tol, f"call {call}, sequence {b} against the oracle: {e:.3e}"
        assert torch.equal(outs[0], outs[1])          # same inputs, same schedule: same bits
    finally:
        layer.close()


def test_static_workspace_refuses_a_shape_beyond_its_maximum():
    layer = SlimLayer(4096, 32, 128, 1.0e6, "bf16", 16, 64, DEV)
    try:
        assert B.slim_workspace_bytes(layer.ctx, 16, 64) > B.slim_static_workspace_max()
        layer.set_wkv(np.eye(4096))
        q = torch.zeros((16, 4096), dtype=torch.bfloat16, device=DEV)
        ld = torch.full((16,), 64, dtype=torch.int32, device=DEV)
        o = torch.full((16, 4096), 7.0, dtype=torch.float32, device=DEV)
        with pytest.raises(B.SlimError) as ei:
            with torch.cuda.device(DEV):
                B.slim_decode_static_ws(layer.ctx, q, layer.cache, ld, o, torch.cuda.current_stream().cuda_stream)
        assert ei.value.status == B.SLIM_ERR_STATIC_WS
        assert "static" in str(ei.value)
        torch.cuda.synchronize()
        assert torch.all(o == 7.0)                      # nothing ran
    finally:
        layer.close()
