"""slim_decode_static_ws: the decode entry point for callers that are not allowed to
allocate device memory (a serving loop with a frozen memory pool, a plug-in on a device
it does not own).  Its scratch is a fixed array inside the library, so the test checks
that it gives the same output as slim_decode with a caller-owned workspace -- twice in
a row, because the second call starts from whatever the first left in the shared array --
and that a shape whose scratch need is above the built-in maximum is refused before
anything is launched.  Collected last on purpose (file name)."""
import numpy as np
import pytest
import torch

from paper_2503_05840_b200 import binding as B
from paper_2503_05840_b200 import synth
from paper_2503_05840_b200.layer import SlimLayer, to_device_keys

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.mark.parametrize("d,H,d_k,theta,dtype,tol", [
    (512, 4, 128, 1.0e4, "bf16", 2e-2),     # tensor-core path
    (384, 6, 64, 0.0, "f32", 1e-4),         # CUDA-core path
])
def test_static_workspace_decode_matches_decode_twice(d, H, d_k, theta, dtype, tol):
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
        for call in range(2):
            o = torch.full((3, d), float("nan"), dtype=torch.float32, device=DEV)
            with torch.cuda.device(DEV):
                B.slim_decode_static_ws(layer.ctx, q, layer.cache, ld, o, stream)
            assert layer.device_status() == B.SLIM_OK
            assert torch.isfinite(o).all(), f"call {call}"
            rms = want.pow(2).mean(dim=1, keepdim=True).sqrt()
            if dtype == "bf16":
                err = ((o - want).abs() / rms).max().item()
            else:
                err = ((o - want).abs() / torch.maximum(want.abs(), rms)).max().item()
            assert err <= tol, f"call {call}: {err:.3e}"
            # different q in between, so the second call really recomputes over stale scratch
            if call == 0:
                other = torch.empty_like(o)
                with torch.cuda.device(DEV):
                    B.slim_decode_static_ws(layer.ctx, torch.flip(q, dims=[0]).contiguous(), layer.cache, ld, other, stream)
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
