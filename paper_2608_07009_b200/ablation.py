"""Cache-policy ablation on a selection trace (the experiment of the paper's Sec. 4.3 / Fig. 6).

Every configuration replays the IDENTICAL selection stream, so differences are replacement decisions alone:
top-k-only staging (B = k), FIFO / random / LRU at B = 2k, LRU at B = 4k run on the GPU through the library's
policy switch in metadata-only mode (no record is fetched), and the offline farthest-next-use policy (Belady),
which needs the future and therefore runs on the host.  The paper's own trace (LongBenchV2 selections of
GLM-5.1) is not available; the seeded synthetic traces of `inputs` stand in for it, so the absolute miss rates
differ from the paper's and only the ordering of the policies is comparable.

    python -m paper_2608_07009_b200.ablation [--workload c2] [--requests 4] [--steps 128]
"""
from __future__ import annotations

import argparse
import json

import numpy as np


def belady_misses(rows: np.ndarray, cache_slots: int) -> np.ndarray:
    """Per-step misses of the offline policy that evicts the resident positions whose next selection lies
    farthest in the future.  rows: int [steps][k], -1 = padding; a selected position equal to -2 - x never occurs."""
    steps = rows.shape[0]
    INF = steps + 1
    nxt = np.full(rows.shape, INF, dtype=np.int64)
    last_seen = {}
    for t in range(steps - 1, -1, -1):
        for j, p in enumerate(rows[t].tolist()):
            if p >= 0:
                nxt[t, j] = last_seen.get(p, INF)
        for p in rows[t].tolist():
            if p >= 0:
                last_seen[p] = t
    resident = {}                       # position -> step of its next selection
    out = np.zeros(steps, dtype=np.int64)
    for t in range(steps):
        cur = {p: int(nxt[t, j]) for j, p in enumerate(rows[t].tolist()) if p >= 0}
        miss = [p for p in cur if p not in resident]
        out[t] = len(miss)
        need = len(resident) + len(miss) - cache_slots
        if need > 0:
            cands = sorted(((nu, p) for p, nu in resident.items() if p not in cur), reverse=True)
            for _, p in cands[:need]:
                del resident[p]
        resident.update(cur)
    return out


def gpu_misses(w, rows_by_step, appended_by_step, cache_slots: int, policy: int, seed: int = 1) -> np.ndarray:
    """Total misses per step over all requests and groups, from the CUDA path in metadata-only mode."""
    import torch
    from . import hisparse as hs
    E = 16
    cap = w.capacity
    hist = [hs.HostHistory(w.num_layers, cap[r], E) for r in range(w.num_requests)]
    gpu = hs.HiSparse(w.num_requests, w.num_layers, w.layers_per_group, cache_slots, w.top_k, E, cap, w.init_len, hist,
                      flags=hs.FLAG_SKIP_IO, policy=policy, policy_seed=seed)
    dev = torch.device("cuda:0")
    kv = torch.zeros((w.num_requests, w.num_layers, E), dtype=torch.uint8, device=dev)
    out = np.zeros(len(rows_by_step), dtype=np.int64)
    acc = torch.zeros(w.num_requests, dtype=torch.int64, device=dev)
    for t, (sel, app) in enumerate(zip(rows_by_step, appended_by_step)):
        if app:
            gpu.append(kv)
        sel_d = torch.from_numpy(sel).to(dev)
        acc.zero_()
        for g in range(w.num_groups):
            _, _, m = gpu.resolve(g * w.layers_per_group, sel_d[g])
            acc += m
        out[t] = int(acc.sum().item())
    assert gpu.status() == 0
    gpu.close()
    for h in hist:
        h.free()
    return out


def main():
    from . import hisparse as hs, inputs
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="c2", choices=["c1", "c2", "c5"])
    ap.add_argument("--requests", type=int, default=4)
    ap.add_argument("--layers", type=int, default=2)
    ap.add_argument("--steps", type=int, default=128)
    ap.add_argument("--skip", type=int, default=16, help="leading steps left out of the means (cold cache)")
    args = ap.parse_args()
    if args.workload == "c1":
        w = inputs.c1_tiny_dsa()
        w.steps = args.steps
    elif args.workload == "c2":
        w = inputs.c2_dsa_decode(num_requests=args.requests, num_layers=args.layers, steps=args.steps)
    else:
        w = inputs.c5_quest_pages(num_requests=args.requests, num_layers=args.layers, steps=args.steps)
    tr = inputs.Trace(w)
    rows, apps = [], []
    for _ in range(args.steps):
        sel, app, _ = tr.step()
        rows.append(sel)
        apps.append(app)
    tr.close()
    k = w.top_k
    valid = sum(int((s >= 0).sum()) for s in rows[args.skip:])
    configs = [("swap-vanilla (B=k)", k, hs.POLICY_LRU), ("fifo (B=2k)", 2 * k, hs.POLICY_FIFO),
               ("random (B=2k)", 2 * k, hs.POLICY_RANDOM), ("lru (B=2k)", 2 * k, hs.POLICY_LRU),
               ("lru (B=4k)", 4 * k, hs.POLICY_LRU)]
    result = {"workload": w.name, "requests": w.num_requests, "groups": w.num_groups, "top_k": k, "steps": args.steps,
              "skipped_steps": args.skip, "miss_rate": {}}
    for name, B, pol in configs:
        if B > hs.MAX_CACHE_SLOTS:
            continue
        m = gpu_misses(w, rows, apps, B, pol)
        result["miss_rate"][name] = float(m[args.skip:].sum() / valid)
    for mult in (2, 4):
        tot = 0
        for g in range(w.num_groups):
            for r in range(w.num_requests):
                tot += int(belady_misses(np.stack([s[g, r] for s in rows]), mult * k)[args.skip:].sum())
        result["miss_rate"]["belady offline (B=%dk)" % mult] = tot / valid
    print(json.dumps(result))


if __name__ == "__main__":
    main()
