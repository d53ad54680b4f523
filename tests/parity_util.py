"""GPU-vs-oracle comparison of block-wise prefill, shared by the GPU tests, the smoke check and the
full-size sampled checks.  Compares, per block and per layer: attention output, log-sum-exp, scores
of all candidates, the retained index set and the retained K/V rows (bit-exact)."""
from __future__ import annotations

import numpy as np
import torch

from oracle.kvc_oracle import KVCOracle

GAP_RTOL = 1e-3          # retained sets must agree bit-exactly when the cut-off gap exceeds this


def tolerances(dtype):
    # attention output / lse absolute tolerances: 1e-4 in fp32, 2e-2 in bf16
    return (1e-4, 1e-4) if dtype == torch.float32 else (2e-2, 2e-3)


def compare_chunk(kvc, orc, layer, q, k, v, pos0, kv_heads=None, teacher_forced=False, out_gpu=None,
                  slot=None, run_gpu=True, n_proxy=0):
    """Runs one block on both sides (or only the oracle if run_gpu is False and out_gpu is given) and
    asserts parity.  Returns a dict of error statistics."""
    cfg = kvc.cfg
    G = cfg.n_q_heads // cfg.n_kv_heads
    heads = list(range(cfg.n_kv_heads)) if kv_heads is None else list(kv_heads)
    n = q.shape[0]
    dev = kvc.device
    Kc, Vc, Pc, len_before = kvc.cache_view(layer)
    if teacher_forced:
        for g in heads:                       # GPU cache <- oracle state (same length by construction)
            L = orc.cache_len(layer, g)
            assert L == len_before
            Kc[g, :L] = torch.from_numpy(orc.K[layer][g]).to(dev).to(kvc.dtype)
            Vc[g, :L] = torch.from_numpy(orc.V[layer][g]).to(dev).to(kvc.dtype)
            Pc[g, :L] = torch.from_numpy(orc.pos[layer][g]).to(dev).to(torch.int32)
    pos_before = Pc[:, :len_before].cpu().numpy().astype(np.int64)
    if run_gpu and n_proxy:
        out_gpu = kvc.prefill_chunk_proxy(layer, q.to(dev), k.to(dev), v.to(dev), n_proxy, pos0)
    elif run_gpu:
        out_gpu = kvc.prefill_chunk(layer, q.to(dev), k.to(dev), v.to(dev), pos0)
    res = orc.prefill_chunk(layer, q.double().numpy(), k.double().numpy(), v.double().numpy(), pos0,
                            kv_heads=kv_heads, n_proxy=n_proxy)
    torch.cuda.synchronize()
    assert kvc.status() == 0, kvc.last_error()
    atol_out, atol_lse = tolerances(kvc.dtype)
    qh = [g * G + hh for g in heads for hh in range(G)]
    out_np = out_gpu.double().cpu().numpy()
    ref = res.out[:, qh]
    assert np.isfinite(out_np[:, qh]).all()
    # max-abs tolerance; a bf16 result cannot be closer than half an ulp (2^-9 relative), which exceeds
    # 2e-2 once |x| > 5.1, so elements with |ref| > 4 are held to the same bound relative to |ref| / 4
    err_el = np.abs(out_np[:, qh] - ref) / np.maximum(1.0, np.abs(ref) / 4.0)
    err_out = err_el.max()
    assert err_out <= atol_out, f"attention output max-abs error {err_out} > {atol_out} (layer {layer}, pos0 {pos0})"
    slot = kvc.slot_of(layer) if slot is None else slot
    lse_gpu, score_gpu = kvc.workspace_view(slot)
    err_lse = np.abs(lse_gpu[:n].double().cpu().numpy()[:, qh] - res.lse[:, qh]).max()
    assert err_lse <= atol_lse, f"lse error {err_lse}"
    stats = dict(err_out=float(err_out), err_lse=float(err_lse), err_score=0.0, adopted=0)

    Kc, Vc, Pc, len_after = kvc.cache_view(layer)
    B = cfg.budget
    assert len_after == min(len_before + n - n_proxy, B)
    for g in heads:
        assert orc.cache_len(layer, g) == len_after
        pos_gpu = Pc[g, :len_after].cpu().numpy().astype(np.int64)
        assert len(np.unique(pos_gpu)) == len_after, "duplicate positions in the cache"
        if res.evicted:
            w = 0 if n_proxy else min(cfg.obs_window if cfg.obs_window else 32, n)   # proxies: nothing is protected
            n_cand = len_before + n - n_proxy - w
            # candidate j of the GPU (physical order before compaction) has position:
            phys_pos = np.concatenate([pos_before[g], pos0 + np.arange(n)])[:n_cand]
            sg = score_gpu[g, :n_cand].double().cpu().numpy()
            so = dict(zip(res.cand_pos[g].tolist(), res.score[g].tolist()))
            so_phys = np.array([so[p] for p in phys_pos.tolist()])
            tol_s = (1e-5 if kvc.dtype == torch.float32 else 2e-4) * max(1.0, so_phys.max())
            err_s = np.abs(sg - so_phys).max()
            stats["err_score"] = max(stats["err_score"], float(err_s))
            assert err_s <= tol_s + 1e-4 * np.abs(so_phys).max(), f"score error {err_s} (kv-head {g})"
            ret_o = res.retained_pos[g]
            ret_g = np.sort(pos_gpu)
            if not np.array_equal(ret_g, ret_o):
                # only legal at a near-tie: every kept candidate must score within GAP_RTOL of the cut-off
                assert res.gap[g] is not None and res.gap[g] <= GAP_RTOL, \
                    f"retained sets differ although the cut-off gap is {res.gap[g]}"
                cand = set(res.cand_pos[g].tolist())
                kept_c = [p for p in ret_g.tolist() if p in cand]
                drop_c = [p for p in cand if p not in set(ret_g.tolist())]
                assert len(kept_c) == B - w
                protected = set(range(pos0 + n - n_proxy - w, pos0 + n - n_proxy))
                assert protected <= set(ret_g.tolist())
                cutoff = min(so[p] for p in (set(ret_o.tolist()) & cand))
                assert min(so[p] for p in kept_c) >= max(so[p] for p in drop_c) - GAP_RTOL * abs(cutoff)
                orc.force_retained(layer, g, ret_g)
                stats["adopted"] += 1
        # retained rows are bit-exact copies of the inputs: compare against the oracle's rows by position
        order = np.argsort(pos_gpu, kind="stable")
        assert np.array_equal(pos_gpu[order], orc.pos[layer][g])
        Kg = Kc[g, :len_after].double().cpu().numpy()[order]
        Vg = Vc[g, :len_after].double().cpu().numpy()[order]
        assert np.array_equal(Kg, orc.K[layer][g]) and np.array_equal(Vg, orc.V[layer][g]), "cache rows are not exact copies"
    return stats


def make_oracle(cfg, n_layers=None, policy="attn") -> KVCOracle:
    return KVCOracle(cfg.n_layers if n_layers is None else n_layers, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim,
                     cfg.budget, cfg.obs_window, policy=policy)


def run_workload_parity(kvc, wl_cfg, layer_tensors, layers, kv_heads=None, teacher_forced=False, chunks=None,
                        policy="attn"):
    """Free-running (or teacher-forced) parity over a whole chunk schedule for the given layers."""
    orc = make_oracle(wl_cfg, policy=policy)
    worst = dict(err_out=0.0, err_lse=0.0, err_score=0.0, adopted=0)
    for pos0, n in (wl_cfg.chunks() if chunks is None else chunks):
        for layer in layers:
            q, k, v = layer_tensors[layer]
            s = compare_chunk(kvc, orc, layer, q[pos0:pos0 + n], k[pos0:pos0 + n], v[pos0:pos0 + n], pos0,
                              kv_heads=kv_heads, teacher_forced=teacher_forced)
            for key in ("err_out", "err_lse", "err_score"):
                worst[key] = max(worst[key], s[key])
            worst["adopted"] += s["adopted"]
    return worst
