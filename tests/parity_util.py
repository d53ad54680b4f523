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


# ------------------------------------------------------------------------------------------------
# Guard regions: every buffer the library writes to or reads from in a parity run (cache blobs, workspace, q, k, v,
# out) sits between two poisoned regions, which are checked after every call.  A store that strays outside a buffer
# (a tile store near the end of a blob, an output row past n, a score past cap) shows up as a changed guard byte.

GUARD_BYTES = 8192
POISON = 0xA5


def _guarded_bytes(nbytes, device):
    """(whole, view): `view` is `nbytes` bytes, 256-byte aligned, with GUARD_BYTES of poison on either side."""
    body = (nbytes + 255) // 256 * 256
    whole = torch.full((GUARD_BYTES + body + GUARD_BYTES,), POISON, dtype=torch.uint8, device=device)
    return whole, whole[GUARD_BYTES:GUARD_BYTES + nbytes]


def guarded_copy(t, device):
    """A device copy of tensor `t` between guard regions: (whole buffer, tensor view)."""
    nbytes = t.numel() * t.element_size()
    whole, view = _guarded_bytes(nbytes, device)
    out = view.view(t.dtype).view(t.shape)
    out.copy_(t)
    return whole, out


def install_guards(kvc):
    """Moves the context's cache blobs and workspace into guarded buffers: poison before the first blob, between
    consecutive blobs, after the last one, and around the workspace.  Only for a context that has not run yet."""
    L, blob = kvc.cfg.n_layers, kvc.blob_bytes
    stride = (blob + 255) // 256 * 256 + GUARD_BYTES
    whole_c = torch.full((GUARD_BYTES + L * stride,), POISON, dtype=torch.uint8, device=kvc.device)
    kvc.cache = whole_c[GUARD_BYTES:].view(L, stride)[:, :blob]
    whole_w, kvc.workspace = _guarded_bytes(kvc.ws_bytes, kvc.device)
    kvc.workspace_init()
    kvc.reset()
    kvc._guards = dict(cache=whole_c, stride=stride, workspace=whole_w)


def check_guards(kvc, extra=()):
    """Asserts that no guard byte around the cache blobs, the workspace and the `extra` (whole, view) pairs changed."""
    g = getattr(kvc, "_guards", None)
    if g is not None:
        whole_c, stride, blob = g["cache"], g["stride"], kvc.blob_bytes
        assert bool((whole_c[:GUARD_BYTES] == POISON).all()), "bytes before the first cache blob were overwritten"
        gaps = whole_c[GUARD_BYTES:].view(kvc.cfg.n_layers, stride)[:, blob:]
        assert bool((gaps == POISON).all()), "bytes after a cache blob were overwritten"
        w = g["workspace"]
        assert bool((w[:GUARD_BYTES] == POISON).all()) and bool((w[GUARD_BYTES + (kvc.ws_bytes + 255) // 256 * 256:] == POISON).all()), \
            "bytes around the workspace were overwritten"
    for whole, view in extra:
        nbytes = view.numel() * view.element_size()
        body = (nbytes + 255) // 256 * 256
        assert bool((whole[:GUARD_BYTES] == POISON).all()) and bool((whole[GUARD_BYTES + body:] == POISON).all()), \
            "bytes around a q / k / v / out buffer were overwritten"
        assert bool((whole[GUARD_BYTES + nbytes:GUARD_BYTES + body] == POISON).all()), "bytes right after a buffer were overwritten"


def pre_state(kvc, layer):
    """What compare_chunk needs to know about a layer's cache BEFORE the GPU runs the block: the positions of
    its entries in physical order and its length."""
    _, _, Pc, len_before = kvc.cache_view(layer)
    return Pc[:, :len_before].cpu().numpy().astype(np.int64), len_before


def compare_chunk(kvc, orc, layer, q, k, v, pos0, kv_heads=None, teacher_forced=False, out_gpu=None,
                  slot=None, pre=None, n_proxy=0):
    """Runs one block on both sides and asserts parity.  If the caller has already run the GPU side (for instance
    as one layer of a layer-batched call) it passes that layer's `out_gpu`, the `pre_state` taken before the
    call and the workspace `slot` the layer used; only the oracle runs here then.  Returns error statistics."""
    cfg = kvc.cfg
    G = cfg.n_q_heads // cfg.n_kv_heads
    heads = list(range(cfg.n_kv_heads)) if kv_heads is None else list(kv_heads)
    n = q.shape[0]
    dev = kvc.device
    if pre is None:
        if not hasattr(kvc, "_guards") and kvc.launch_count() == 0 and kvc.cache is not None:
            install_guards(kvc)                   # first use of this context: put its buffers between guard regions
        Kc, Vc, Pc, len_before = kvc.cache_view(layer)
        if teacher_forced:
            for g in heads:                       # GPU cache <- oracle state (same length by construction)
                L = orc.cache_len(layer, g)
                assert L == len_before
                Kc[g, :L] = torch.from_numpy(orc.K[layer][g]).to(dev).to(kvc.dtype)
                Vc[g, :L] = torch.from_numpy(orc.V[layer][g]).to(dev).to(kvc.dtype)
                Pc[g, :L] = torch.from_numpy(orc.pos[layer][g]).to(dev).to(torch.int32)
        pos_before = Pc[:, :len_before].cpu().numpy().astype(np.int64)
        bufs = [guarded_copy(t, dev) for t in (q, k, v)] + [guarded_copy(torch.zeros_like(q), dev)]
        (qd, kd, vd, od) = [b[1] for b in bufs]
        if n_proxy:
            out_gpu = kvc.prefill_chunk_proxy(layer, qd, kd, vd, n_proxy, pos0, od)
        else:
            out_gpu = kvc.prefill_chunk(layer, qd, kd, vd, pos0, od)
        torch.cuda.synchronize()
        check_guards(kvc, bufs)
        assert torch.equal(qd.cpu(), q.cpu()) and torch.equal(kd.cpu(), k.cpu()) and torch.equal(vd.cpu(), v.cpu()), "an input was modified"
    else:
        assert out_gpu is not None and not teacher_forced
        pos_before, len_before = pre
    res = orc.prefill_chunk(layer, q.double().numpy(), k.double().numpy(), v.double().numpy(), pos0,
                            kv_heads=kv_heads, n_proxy=n_proxy)
    torch.cuda.synchronize()
    assert kvc.status() == 0, kvc.last_error()
    atol_out, atol_lse = tolerances(kvc.dtype)
    qh = [g * G + hh for g in heads for hh in range(G)]
    out_np = out_gpu.double().cpu().numpy()
    ref = res.out[:, qh]
    assert np.isfinite(out_np[:, qh]).all()
    # Plain max-abs tolerance.  A bf16 result is a multiple of its ulp, and from |x| = 4 on that ulp (2^-5) is
    # larger than 2e-2, so a correctly rounded output can already miss the bound there.  The only escape allowed:
    # a bf16 element may instead lie within one bf16 ulp of the oracle value rounded to bf16.  Both the plain
    # max-abs and the number of elements that needed the escape are reported.
    err_el = np.abs(out_np[:, qh] - ref)
    err_out = float(err_el.max())
    n_escaped = 0
    over = err_el > atol_out
    if over.any():
        assert kvc.dtype == torch.bfloat16, f"attention output max-abs error {err_out} > {atol_out} (layer {layer}, pos0 {pos0})"
        ref_over = ref[over]
        ref_bf16 = torch.from_numpy(ref_over).to(torch.bfloat16).double().numpy()
        ulp = 2.0 ** (np.floor(np.log2(np.maximum(np.abs(ref_bf16), 2.0 ** -126))) - 7)
        bad = np.abs(out_np[:, qh][over] - ref_bf16) > ulp
        assert not bad.any(), (f"attention output: {int(bad.sum())} elements off by more than {atol_out} and more than one bf16 "
                               f"ulp from the rounded oracle value; max-abs {err_out} (layer {layer}, pos0 {pos0})")
        n_escaped = int(over.sum())
    slot = kvc.slot_of(layer) if slot is None else slot
    lse_gpu, score_gpu = kvc.workspace_view(slot)
    err_lse = np.abs(lse_gpu[:n].double().cpu().numpy()[:, qh] - res.lse[:, qh]).max()
    assert err_lse <= atol_lse, f"lse error {err_lse}"
    stats = dict(err_out=float(err_out), err_lse=float(err_lse), err_score=0.0, adopted=0, ulp_escapes=n_escaped,
                 max_abs_ref=float(np.abs(ref).max()))

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


def assert_output_bound(worst, dtype):
    """The summary of a run obeys the output tolerance: plain max-abs within 1e-4 (fp32) / 2e-2 (bf16); a larger
    bf16 maximum is possible only through elements that compare_chunk passed by the one-ulp rule."""
    atol = tolerances(dtype)[0]
    assert worst["err_out"] <= atol or (dtype == torch.bfloat16 and worst["ulp_escapes"] > 0), worst


def make_oracle(cfg, n_layers=None, policy="attn") -> KVCOracle:
    return KVCOracle(cfg.n_layers if n_layers is None else n_layers, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim,
                     cfg.budget, cfg.obs_window, policy=policy)


def run_workload_parity(kvc, wl_cfg, layer_tensors, layers, kv_heads=None, teacher_forced=False, chunks=None,
                        policy="attn"):
    """Free-running (or teacher-forced) parity over a whole chunk schedule for the given layers."""
    orc = make_oracle(wl_cfg, policy=policy)
    worst = dict(err_out=0.0, err_lse=0.0, err_score=0.0, adopted=0, ulp_escapes=0, max_abs_ref=0.0)
    for pos0, n in (wl_cfg.chunks() if chunks is None else chunks):
        for layer in layers:
            q, k, v = layer_tensors[layer]
            s = compare_chunk(kvc, orc, layer, q[pos0:pos0 + n], k[pos0:pos0 + n], v[pos0:pos0 + n], pos0,
                              kv_heads=kv_heads, teacher_forced=teacher_forced)
            for key in ("err_out", "err_lse", "err_score", "max_abs_ref"):
                worst[key] = max(worst[key], s[key])
            worst["adopted"] += s["adopted"]
            worst["ulp_escapes"] += s["ulp_escapes"]
    print(f"parity {wl_cfg.name}: plain max-abs out {worst['err_out']:.3e} (max |ref| {worst['max_abs_ref']:.2f}, "
          f"{worst['ulp_escapes']} elements passed by the one-ulp rule), lse {worst['err_lse']:.3e}, "
          f"score {worst['err_score']:.3e}, near-tie sets adopted {worst['adopted']}")
    return worst
