"""One context split into slices, as several GPUs would hold it, through the C ABI: every slice gets its
own cache and a slim_decode_partial call (run one after the other on this GPU -- the calls do not wait
on each other), the stacked results go through slim_combine_project.  Checked against the oracle's
partials, against the oracle on the whole context, and against slim_decode on one whole cache."""
import numpy as np
import pytest
import torch

from oracle import slim_oracle as so
from paper_2503_05840_b200 import binding as B
from paper_2503_05840_b200 import context_split as cs
from paper_2503_05840_b200 import synth
from paper_2503_05840_b200.layer import SlimLayer, to_device_keys

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.mark.parametrize("d,H,d_k,theta,dtype,world,ramp", [(512, 4, 128, 1.0e6, "bf16", 3, False), (1280, 20, 64, 0.0, "bf16", 2, False),
                                                            (384, 6, 64, 1.0e4, "f32", 4, False), (384, 4, 96, 1.0e4, "bf16", 8, False),
                                                            (512, 4, 128, 1.0e4, "bf16", 2, True)])
def test_split_context_joins_to_the_whole(d, H, d_k, theta, dtype, world, ramp):
    lengths = np.array([1000, 333, 0, 17, 5], dtype=np.int32)
    batch, t_cap = len(lengths), 1000
    cfg = synth.SlimConfig("split", d, H, d_k, batch, t_cap, 1, theta, dtype)
    L = synth.make_layer(cfg, 97, lengths=lengths)
    if ramp:      # keys that grow along the context: arguments far above a unit's first tile, so slices take the exact redo
        L.K[0] = synth.round_to_bf16(L.K[0] * (1.0 + 0.3 * np.arange(t_cap, dtype=np.float32)[:, None]))
    W_KV = so.oracle_wkv(L.W_K, L.W_V)
    whole = SlimLayer(d, H, d_k, theta, dtype, batch, t_cap, DEV)
    slices = []
    try:
        Kd = to_device_keys(L.K, dtype, DEV)
        q = to_device_keys(L.q, dtype, DEV)
        ld = torch.from_numpy(lengths).to(DEV)
        whole.k.copy_(Kd); whole.set_wkv(W_KV)
        want = whole.decode(q, ld).clone()
        st = torch.cuda.current_stream().cuda_stream
        q_pos = (ld - 1).clamp(min=0).to(torch.int32)
        lse_all = torch.full((world, batch, H), float("nan"), dtype=torch.float32, device=DEV)
        u_all = torch.full((world, batch, H, d), float("nan"), dtype=torch.float32, device=DEV)
        tol = 2e-2 if dtype == "bf16" else 1e-4
        for r in range(world):
            first, count = cs.shard_batch(lengths, world, r)
            cap = max(max(count), 16)
            lay = SlimLayer(d, H, d_k, theta, dtype, batch, cap, DEV)
            slices.append(lay)
            lay.set_wkv(W_KV)
            B.slim_reserve_positions(lay.ctx, t_cap + 16)             # positions of the whole context, not of the slice
            lay.k.fill_(float("nan"))
            for b in range(batch):
                a = first[b] * cs.TILE
                lay.k[b, :count[b]] = Kd[b, a:a + count[b]]
            with torch.cuda.device(DEV):
                B.slim_decode_partial(lay.ctx, q, lay.cache, torch.tensor(count, dtype=torch.int32, device=DEV),
                                      torch.tensor(first, dtype=torch.int32, device=DEV), q_pos, lse_all[r], u_all[r], lay.workspace, st)
            assert lay.device_status() == B.SLIM_OK
            lse_r, u_r = lse_all[r].cpu().numpy().astype(np.float64), u_all[r].cpu().numpy().astype(np.float64)
            for b in range(batch):
                a = first[b] * cs.TILE
                lse_o, u_o = so.oracle_slim_partial(L.q[b], L.K[b, a:a + count[b]], a, int(lengths[b]) - 1, H, theta)
                if count[b] == 0:
                    assert np.all(np.isneginf(lse_r[b]))
                    continue
                assert np.max(np.abs(lse_r[b] - lse_o)) <= 2e-3, f"rank {r} seq {b}: lse"
                for h in range(H):
                    e = so.err_rms_norm(u_r[b, h], u_o[h]) if dtype == "bf16" else so.err_fp32_norm(u_r[b, h], u_o[h])
                    assert e <= tol, f"rank {r} seq {b} head {h}: {e:.3e}"
        o = torch.full((batch, d), float("nan"), dtype=torch.float32, device=DEV)
        with torch.cuda.device(DEV):
            # rank order is free: hand the slices over reversed
            B.slim_combine_project(whole.ctx, lse_all.flip(0).contiguous(), u_all.flip(0).contiguous(), world, ld, batch, o, whole.workspace, st)
        assert whole.device_status() == B.SLIM_OK
        got = o.cpu().numpy().astype(np.float64)
        ref = so.oracle_slim_batch(L.q, L.K, lengths, W_KV, H, theta)
        for b in range(batch):
            if lengths[b] == 0:
                assert np.all(got[b] == 0)
                continue
            e = so.err_rms_norm(got[b], ref[b]) if dtype == "bf16" else so.err_fp32_norm(got[b], ref[b])
            assert e <= tol, f"seq {b}: {e:.3e}"
        rms = want.pow(2).mean(dim=1, keepdim=True).sqrt().clamp(min=1e-30)
        assert ((o - want).abs() / rms).max().item() <= tol          # and the one-GPU result
    finally:
        whole.close()
        for lay in slices:
            lay.close()


def test_split_positions_outside_the_reserved_table_are_reported():
    lay = SlimLayer(256, 2, 128, 1.0e4, "bf16", 1, 64, DEV)
    try:
        lay.set_wkv(np.eye(256))
        q = torch.zeros((1, 256), dtype=torch.bfloat16, device=DEV)
        lse = torch.empty((1, 2), dtype=torch.float32, device=DEV); u = torch.empty((1, 2, 256), dtype=torch.float32, device=DEV)
        one = torch.tensor([64], dtype=torch.int32, device=DEV)
        with torch.cuda.device(DEV):
            B.slim_decode_partial(lay.ctx, q, lay.cache, one, torch.tensor([1000], dtype=torch.int32, device=DEV),
                                  torch.tensor([20000], dtype=torch.int32, device=DEV), lse, u, lay.workspace,
                                  torch.cuda.current_stream().cuda_stream)
        assert lay.device_status() == B.SLIM_ERR_CAPACITY           # clamped into the table, nothing read outside it
    finally:
        lay.close()
