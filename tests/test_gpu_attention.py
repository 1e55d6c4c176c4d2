"""The sparse-attention consumer (hisparse_sparse_attention, through the C-ABI binding) against the fp64 oracle
(oracle/attention_oracle.py), on slot tables that the library's own resolve emitted and on hand-made ones.

Tolerance: inputs are bf16 on both sides, so products are exact; the kernel accumulates in
fp32 and rounds the softmax weights to bf16 (relative error 2^-9 each) before they multiply the values, and its
normaliser is the sum of the unrounded weights.  out is a convex combination of the values, so
|out - exact| <= 1e-2 * max |value| elementwise; lse is fp32 arithmetic on scores of a few units: 2e-3 absolute.
"""
import numpy as np
import pytest
import torch

from oracle import Oracle
from oracle.attention_oracle import f32_to_bf16, bf16_to_f64, sparse_attention
from paper_2608_07009_b200 import HiSparse, HostHistory, HiSparseError, inputs, hisparse as hs

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def bf16_history(rng, L, cap, D):
    """A host history whose records are D bf16 numbers ~ N(0, 1)."""
    return f32_to_bf16(rng.standard_normal((L, cap, D)).astype(np.float32)).view(np.uint8).reshape(L, cap, 2 * D)


def check(out, lse, out_ref, lse_ref, vmax):
    out, lse = out.cpu().numpy().astype(np.float64), lse.cpu().numpy().astype(np.float64)
    assert np.all(np.abs(out - out_ref) <= 1e-2 * vmax), float(np.abs(out - out_ref).max())
    fin = np.isfinite(lse_ref)
    assert np.array_equal(np.isneginf(lse), ~fin)
    assert np.all(np.abs(lse[fin] - lse_ref[fin]) <= 2e-3), float(np.abs(lse[fin] - lse_ref[fin]).max())


@pytest.mark.parametrize("N,H,D,DV,k,B,steps", [
    (3, 16, 576, 512, 256, 512, 3),       # the DSA record: 512-number latent + 64-number rotary key
    (2, 32, 576, 512, 70, 128, 2),        # two head groups, a ragged last tile
    (5, 16, 144, 128, 33, 64, 2),         # small records (an odd number of k-steps), one entry past a tile
    (1, 16, 256, 256, 512, 1024, 2),      # value = the whole record; many splits for one request
])
def test_attention_over_resolved_tables_matches_the_oracle(N, H, D, DV, k, B, steps):
    rng = np.random.default_rng(N * 1000 + k)
    E, ctx = 2 * D, 4 * B
    w = inputs.Workload("att", inputs.KIND_DSA_MIX, N, 1, 1, k, B, E, [ctx] * N, steps + 1, append_every=1 << 30,
                        keep=(3 * k) // 4, recent_window=64, seed=5, config_id=13)
    cap = w.capacity
    hist, hist_cpu = [], []
    for r in range(N):
        h = HostHistory(1, cap[r], E)
        data = bf16_history(rng, 1, cap[r], D)
        h.numpy()[:] = data
        hist.append(h)
        hist_cpu.append(data.copy())
    gpu = HiSparse(N, 1, 1, B, k, E, cap, [ctx] * N, hist)
    orc = Oracle(N, 1, 1, B, k, E, cap, [ctx] * N, hist_cpu)
    tr = inputs.Trace(w)
    scale = 1.0 / np.sqrt(D)
    try:
        for step in range(steps):
            sel, _, _ = tr.step()
            row = np.ascontiguousarray(sel[0])
            if step == steps - 1:
                row = row.copy()
                row[:, ::7] = -1                      # padding in the last step
            tab_o, _, _ = orc.resolve(0, row)
            tab_d, _, _ = gpu.resolve(0, torch.from_numpy(row).to(DEV))
            assert np.array_equal(tab_d.cpu().numpy(), tab_o)
            q = f32_to_bf16(rng.standard_normal((N, H, D)).astype(np.float32))
            q_d = torch.from_numpy(q.view(np.int16)).to(DEV).view(torch.bfloat16)
            out, lse = gpu.sparse_attention(0, q_d, tab_d, DV, scale)
            pool = orc.pool(0).reshape(-1, E)
            out_ref, lse_ref = sparse_attention(pool, tab_o, q, DV, scale)
            vmax = np.abs(bf16_to_f64(pool.reshape(-1).view(np.uint16))).max()
            check(out, lse, out_ref, lse_ref, vmax)
        assert gpu.status() == 0
    finally:
        tr.close()
        gpu.close()
        orc.close()
        for h in hist:
            h.free()


def test_attention_edge_rows_and_placement():
    """All-padding rows give zeros and -inf; a dominant key returns its own value; the same logical records in other
    slots give the same output (placement does not change what attention computes, Sec. 3.1)."""
    rng = np.random.default_rng(9)
    N, H, D, DV, k, B = 2, 16, 128, 128, 64, 64
    E = 2 * D
    hist = [HostHistory(1, 200, E) for _ in range(N)]
    data = [bf16_history(rng, 1, 200, D) for _ in range(N)]
    for h, x in zip(hist, data):
        h.numpy()[:] = x
    gpu = HiSparse(N, 1, 1, B, k, E, [200] * N, [200] * N, hist)
    try:
        sel = np.stack([rng.permutation(200)[:k] for _ in range(N)]).astype(np.int32)
        tab, _, _ = gpu.resolve(0, torch.from_numpy(sel).to(DEV))
        pool = gpu.gather(0, torch.arange(N * k, dtype=torch.int32, device=DEV).view(N, k) // k * (B + 1)
                          + torch.arange(N * k, dtype=torch.int32, device=DEV).view(N, k) % k).cpu().numpy()
        # the oracle's pool: record index r*(B+1)+slot; cold cache fills slots 0..k-1 in selection order
        full = np.zeros((N * (B + 1), E), dtype=np.uint8)
        for r in range(N):
            full[r * (B + 1):r * (B + 1) + k] = pool[r]
            assert np.array_equal(pool[r], data[r][0][sel[r]])
        q = f32_to_bf16(rng.standard_normal((N, H, D)).astype(np.float32))
        rec0 = bf16_to_f64(data[0][0][sel[0, 5]].view(np.uint16))
        q[0, 3] = f32_to_bf16((60.0 * rec0).astype(np.float32))       # head 3 of request 0 locks onto entry 5
        tab_h = tab.cpu().numpy().copy()
        tab_h[1, :] = -1                                               # request 1: nothing selected
        q_d = torch.from_numpy(q.view(np.int16)).to(DEV).view(torch.bfloat16)
        out, lse = gpu.sparse_attention(0, q_d, torch.from_numpy(tab_h).to(DEV), DV, 1.0)
        out_ref, lse_ref = sparse_attention(full, tab_h, q, DV, 1.0)
        check(out, lse, out_ref, lse_ref, np.abs(bf16_to_f64(full.reshape(-1).view(np.uint16))).max())
        assert torch.all(out[1] == 0) and torch.all(torch.isneginf(lse[1]))
        assert np.allclose(out[0, 3].cpu().numpy(), rec0[:DV], atol=1e-2 * np.abs(rec0).max())
        # the same selection in another order lands in other table positions: same outputs
        perm = rng.permutation(k)
        out2, lse2 = gpu.sparse_attention(0, q_d, torch.from_numpy(np.ascontiguousarray(tab_h[:, perm])).to(DEV), DV, 1.0)
        assert torch.allclose(out, out2, atol=2e-2 * float(np.abs(rec0).max())) and torch.allclose(lse[0], lse2[0], atol=4e-3)
        # shapes the kernel does not take are refused before anything is enqueued
        for heads, dv in ((8, 128), (16, 64), (16, 100), (16, 256)):
            with pytest.raises(HiSparseError) as e:
                gpu.attention_workspace_bytes(heads, dv)
            assert e.value.code == hs.EINVAL
    finally:
        gpu.close()
        for h in hist:
            h.free()
    # records longer than 576 numbers: the kernel's query registers are sized for them, anything longer is refused
    hist = [HostHistory(1, 40, 1280)]
    gpu = HiSparse(1, 1, 1, 16, 8, 1280, [40], [40], hist)
    try:
        with pytest.raises(HiSparseError) as e:
            gpu.attention_workspace_bytes(16, 512)
        assert e.value.code == hs.EINVAL
    finally:
        gpu.close()
        hist[0].free()
