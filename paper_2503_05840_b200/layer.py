"""SlimLayer: a convenience owner of the torch buffers one attention layer
needs (key storage, workspace, output).  It only allocates memory and forwards
to the C-ABI calls of the same names; no arithmetic happens here."""
from __future__ import annotations

import numpy as np
import torch

from . import binding as B


class SlimLayer:
    def __init__(self, d: int, H: int, d_k: int, rope_theta: float, dtype: str, batch: int, t_cap: int,
                 device: str = "cuda:0", workspace: "torch.Tensor | None" = None):
        if not torch.cuda.is_available():
            raise RuntimeError("SlimLayer needs a CUDA device (there is no CPU fallback)")
        self.device = torch.device(device)
        self.d, self.H, self.d_k, self.batch, self.t_cap = d, H, d_k, batch, t_cap
        self.dtype = dtype
        # type of q, of new key rows and of W_KV; an "fp8" layer keeps only its cache in 8 bits
        self.tdtype = torch.float32 if dtype == "f32" else torch.bfloat16
        with torch.cuda.device(self.device):
            self.ctx = B.slim_create(d, H, d_k, rope_theta, {"f32": B.SLIM_F32, "bf16": B.SLIM_BF16, "fp8": B.SLIM_FP8}[dtype])
            if dtype == "fp8":     # codes [batch][t_cap][d], then the exponents: filled through append_k only
                self.k = torch.zeros(B.slim_cache_bytes(self.ctx, batch, t_cap), dtype=torch.uint8, device=self.device)
            else:
                self.k = torch.zeros((batch, t_cap, d), dtype=self.tdtype, device=self.device)
            self.cache = B.slim_cache_create(self.ctx, self.k, batch, t_cap)
            need = B.slim_workspace_bytes(self.ctx, batch, t_cap)
            if workspace is None:      # layers that run one after another on a stream may share one
                workspace = torch.empty(need, dtype=torch.uint8, device=self.device)
            assert workspace.numel() >= need and workspace.data_ptr() % 256 == 0
            self.workspace = workspace
            self.o = torch.empty((batch, d), dtype=torch.float32, device=self.device)

    # ---- set-up -------------------------------------------------------------
    def set_weights(self, W_K, W_V, want_wkv: bool = False):
        with torch.cuda.device(self.device):
            return B.slim_set_weights(self.ctx, W_K, W_V, want_wkv)

    def set_wkv(self, W_KV) -> None:
        with torch.cuda.device(self.device):
            B.slim_set_wkv(self.ctx, W_KV)

    def set_path(self, path: int) -> None:
        B.slim_set_path(self.ctx, path)

    def query(self, key: int) -> int:
        return B.slim_query(self.ctx, key)

    # ---- hot path -----------------------------------------------------------
    def append_k(self, k_new: torch.Tensor, positions: torch.Tensor) -> None:
        n_new = k_new.shape[1] if k_new.dim() == 3 else 1
        B.slim_append_k(self.ctx, self.cache, k_new, positions, n_new,
                        torch.cuda.current_stream(self.device).cuda_stream)

    def decode(self, q: torch.Tensor, lengths: torch.Tensor, o: torch.Tensor | None = None) -> torch.Tensor:
        o = self.o if o is None else o
        B.slim_decode(self.ctx, q, self.cache, lengths, o, self.workspace,
                      torch.cuda.current_stream(self.device).cuda_stream)
        return o

    def decode_step(self, q: torch.Tensor, k_new: torch.Tensor, lengths: torch.Tensor,
                    o: torch.Tensor | None = None) -> torch.Tensor:
        o = self.o if o is None else o
        B.slim_decode_step(self.ctx, q, k_new, self.cache, lengths, o, self.workspace,
                           torch.cuda.current_stream(self.device).cuda_stream)
        return o

    def profile(self, enable: bool) -> None:
        B.slim_profile_enable(self.ctx, enable)

    def profile_read(self):
        return B.slim_profile_read(self.ctx)

    def device_status(self) -> int:
        return B.slim_device_status(self.ctx, torch.cuda.current_stream(self.device).cuda_stream)

    def close(self) -> None:
        if getattr(self, "cache", None):
            B.slim_cache_destroy(self.cache); self.cache = None
        if getattr(self, "ctx", None):
            B.slim_destroy(self.ctx); self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def to_device_keys(K_f32: np.ndarray, dtype: str, device) -> torch.Tensor:
    """Host float32 array holding cache-dtype values -> device tensor of the cache dtype (exact)."""
    t = torch.from_numpy(np.ascontiguousarray(K_f32))
    return t.to(device=device, dtype=torch.bfloat16 if dtype == "bf16" else torch.float32)
