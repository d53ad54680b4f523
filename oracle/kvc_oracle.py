"""CPU oracle for block-wise prefill with a budgeted KV cache ("compress as you prefill").

TEST INFRASTRUCTURE ONLY.  This is a plain, slow, fp64 numpy statement of what
the method computes, used to check the CUDA library.  It shares no code with
the CUDA path and must never be imported by it: only tests, the smoke check and
the benchmark's CPU-baseline leg may use this module.

What is computed, per block (Alg. 1 of the paper), independently for every
(layer, kv-head):

  1. append the block's keys/values to the cache                      (Alg. 1, "C <- C u (K_i, V_i)")
  2. attention of the block's queries over cache + block, causal
     inside the block                                                 (Eq. 1)
  3. if |C| > M: importance score of every cached key from the
     attention probabilities of the observer queries                  (Eq. 4)
  4. evict the |C| - M lowest-scoring entries                         (Alg. 1, "Evict(C, k_excess)")
  5. the cache is again M entries                                     (Sec. 3.1)

Readings where the paper is silent (each is a documented choice, see the
design notes of the repository):
  * observers = the block's own last w query rows (observation-window idea of
    the method Eq. 4 is "based on"); their own keys (the last w entries) are
    never evicted;
  * several observer rows and the G query heads sharing a kv-head are combined
    by summation of probabilities;
  * the probabilities are the true attention probabilities of those rows, i.e.
    normalised over everything the row attends to;
  * ties at the cut-off keep the older entry (smaller position);
  * scores are recomputed from scratch at every eviction round;
  * proxy-query variant (Sec. 3.2: the observers are proxy tokens taken from the text prompt): a call
    may carry t trailing proxy tokens.  They attend like any other token of the block (causally, after
    the block's real tokens) and are the observers of the score, but their keys/values never enter the
    cache; there is then no protected window: all |C| entries compete and the M best stay.
  * query-agnostic policy (Sec. 3.2, "Query-Agnostic Eviction"): the anchor mu is the mean of the
    raw keys the cache holds right after the block was appended, "similarity" is the cosine, and
    the score of an entry is 1 - cos(k_j, mu) (so "lower similarity" = higher score = retained);
    the same last-w entries are protected and ties keep the older entry; a zero key or a zero
    anchor has cosine 0.

Pins (tests/test_oracle_pins.py): budget >= sequence length reproduces dense
causal attention (library routine); empty-cache block equals causal attention
on the block; permutation invariance over cache order; probability mass of the
score; one observer / one head reduces to a single softmax row; one block of
the whole sequence reproduces post-prefill compression computed with library
softmax / top-k; brute-force subset enumeration on tiny inputs; tie-break on
duplicated keys; retained rows are bit-identical copies; Eq. 2 byte counts.  Query-agnostic
score: library cosine similarity; an outlier among identical keys is the one kept; invariance
under a common scaling and a common rotation of all keys; brute force.
End-to-end model accuracy (the paper's tables): parity unpinned, it needs
datasets and weights that are not available.
"""
from __future__ import annotations

import dataclasses
from typing import List, Optional

import numpy as np


@dataclasses.dataclass
class ChunkResult:
    out: np.ndarray                      # [n][Hq][d] fp64, Eq. 1
    lse: np.ndarray                      # [n][Hq] fp64, log-sum-exp of the scaled scores of each row
    evicted: bool                        # whether |C| > M triggered (Alg. 1)
    score: List[Optional[np.ndarray]]    # per kv-head: fp64 score of every candidate, in cache order
    cand_pos: List[Optional[np.ndarray]] # per kv-head: position of every candidate, same order
    retained_pos: List[np.ndarray]       # per kv-head: sorted positions in the cache after the block
    gap: List[Optional[float]]           # per kv-head: relative score gap at the cut-off


class KVCOracle:
    """Budgeted KV cache of one model: state is, per (layer, kv-head), a list of (pos, k, v)."""

    def __init__(self, n_layers: int, n_q_heads: int, n_kv_heads: int, head_dim: int,
                 budget: int, obs_window: int = 32, scale: Optional[float] = None, policy: str = "attn"):
        assert n_q_heads % n_kv_heads == 0
        self.L, self.Hq, self.Hkv, self.d = n_layers, n_q_heads, n_kv_heads, head_dim
        self.G = n_q_heads // n_kv_heads
        self.M = budget
        self.obs_window = obs_window
        assert policy in ("attn", "keydiff")
        self.policy = policy
        self.scale = (1.0 / np.sqrt(head_dim)) if scale is None else float(scale)   # Eq. 1: 1/sqrt(d_k)
        self.reset()

    def reset(self):
        """C <- empty (Alg. 1)."""
        self.pos = [[np.zeros(0, dtype=np.int64) for _ in range(self.Hkv)] for _ in range(self.L)]
        self.K = [[np.zeros((0, self.d)) for _ in range(self.Hkv)] for _ in range(self.L)]
        self.V = [[np.zeros((0, self.d)) for _ in range(self.Hkv)] for _ in range(self.L)]

    def cache_len(self, layer: int, g: int = 0) -> int:
        return len(self.pos[layer][g])

    def load_state(self, layer: int, g: int, pos, K, V):
        """Overwrite one (layer, kv-head) cache (used to teacher-force or adopt a valid alternative)."""
        order = np.argsort(np.asarray(pos, dtype=np.int64), kind="stable")
        self.pos[layer][g] = np.asarray(pos, dtype=np.int64)[order]
        self.K[layer][g] = np.asarray(K, dtype=np.float64)[order]
        self.V[layer][g] = np.asarray(V, dtype=np.float64)[order]

    def force_retained(self, layer: int, g: int, keep_pos):
        """Replace the retained set of (layer, g) by ``keep_pos`` (subset of what was present
        before the last eviction): used when two selections are both valid (near-tie at the cut-off)."""
        keep = np.sort(np.asarray(keep_pos, dtype=np.int64))
        allpos, allK, allV = self._pre_evict[layer][g]
        idx = np.searchsorted(allpos, keep)
        assert np.array_equal(allpos[idx], keep), "forced set must come from the pre-eviction cache"
        self.pos[layer][g], self.K[layer][g], self.V[layer][g] = allpos[idx], allK[idx], allV[idx]

    # ------------------------------------------------------------------------------------
    def prefill_chunk(self, layer: int, q, k, v, pos0: int, kv_heads=None, n_proxy: int = 0) -> ChunkResult:
        """One block of Alg. 1 for one layer.  ``kv_heads`` restricts the work to a subset of kv-heads
        (they are independent); the other heads' state and outputs are left untouched (zeros).
        The last ``n_proxy`` rows of q/k/v are proxy query tokens (observers only, never cached)."""
        q = np.asarray(q, dtype=np.float64)
        k = np.asarray(k, dtype=np.float64)
        v = np.asarray(v, dtype=np.float64)
        n = q.shape[0]
        assert q.shape == (n, self.Hq, self.d) and k.shape == (n, self.Hkv, self.d) and v.shape == k.shape
        assert 0 <= n_proxy < n
        n_real = n - n_proxy
        G, M = self.G, self.M
        out = np.zeros((n, self.Hq, self.d))
        lse = np.zeros((n, self.Hq))
        scores, cand_pos, retained, gaps = [], [], [], []
        evicted_any = False
        if not hasattr(self, "_pre_evict"):
            self._pre_evict = [[None] * self.Hkv for _ in range(self.L)]

        for g in range(self.Hkv):
            if kv_heads is not None and g not in kv_heads:
                scores.append(None); cand_pos.append(None); gaps.append(None); retained.append(None)
                continue
            # 1. append (Alg. 1): the block's keys/values join the cache before anything is evicted
            n_c = len(self.pos[layer][g])
            pos = np.concatenate([self.pos[layer][g], pos0 + np.arange(n, dtype=np.int64)])
            K = np.concatenate([self.K[layer][g], k[:, g, :]], axis=0)
            V = np.concatenate([self.V[layer][g], v[:, g, :]], axis=0)
            tot = n_c + n                                   # keys the block's rows can attend to (proxies included)

            # 2. attention (Eq. 1).  Row i sees every older cache entry and block keys t <= i.
            visible = np.ones((n, tot), dtype=bool)
            visible[:, n_c:] = np.tril(np.ones((n, n), dtype=bool))
            P = np.zeros((G, n, tot))                       # probabilities, kept for the score
            for hh in range(G):
                h = g * G + hh                              # consecutive query heads share kv-head g
                S = self.scale * (q[:, h, :] @ K.T)         # softmax argument of Eq. 1
                S = np.where(visible, S, -np.inf)
                m = S.max(axis=1, keepdims=True)
                E = np.exp(S - m)
                l = E.sum(axis=1, keepdims=True)
                lse[:, h] = (m + np.log(l))[:, 0]
                P[hh] = E / l
                out[:, h, :] = P[hh] @ V

            if n_proxy:
                # the proxies' keys/values are not part of the cache: drop them again
                tot = n_c + n_real
                pos, K, V = pos[:tot], K[:tot], V[:tot]
            self._pre_evict[layer][g] = (pos, K, V)
            # Alg. 1: evict only if |C| > M (strict)
            if tot <= M:
                self.pos[layer][g], self.K[layer][g], self.V[layer][g] = pos, K, V
                scores.append(None); cand_pos.append(None); gaps.append(None)
                retained.append(np.sort(pos))
                continue
            evicted_any = True

            # 3. score (Eq. 4): observers = last w rows of the block; candidates = all entries but the
            #    observers' own w keys, which are always kept
            if n_proxy:
                w, n_cand = n_proxy, tot                    # observers = the proxies; every entry competes
            else:
                w = min(self.obs_window, n)
                assert w <= M
                n_cand = tot - w
            if self.policy == "attn":
                score = P[:, n - w:, :n_cand].sum(axis=(0, 1))   # P is over all keys the rows saw: the true normaliser
            else:
                # query-agnostic (Sec. 3.2): anchor = mean of the cached keys, keep the keys least similar to it
                mu = K.mean(axis=0)
                denom = np.linalg.norm(K[:n_cand], axis=1) * np.linalg.norm(mu)
                cos = np.divide(K[:n_cand] @ mu, denom, out=np.zeros(n_cand), where=denom > 0)
                score = 1.0 - cos

            # 4. select: keep the (M - w) candidates that come first under
            #    (score descending, position ascending); evict the other tot - M (Alg. 1)
            n_keep = M - w if not n_proxy else M
            order = np.lexsort((pos[:n_cand], -score))      # primary key: -score, secondary: pos
            keep_c = order[:n_keep]
            if 0 < n_keep < n_cand:
                s_in, s_out = score[order[n_keep - 1]], score[order[n_keep]]
                gaps.append(float((s_in - s_out) / max(abs(s_in), 1e-300)))
            else:
                gaps.append(None)

            # 5. compact: the cache is the retained candidates plus the protected tail, |C| = M
            keep = np.sort(np.concatenate([keep_c, np.arange(n_cand, tot)]))
            assert len(keep) == M
            keep = keep[np.argsort(pos[keep], kind="stable")]
            self.pos[layer][g], self.K[layer][g], self.V[layer][g] = pos[keep], K[keep], V[keep]
            scores.append(score); cand_pos.append(pos[:n_cand].copy())
            retained.append(self.pos[layer][g].copy())

        return ChunkResult(out, lse, evicted_any, scores, cand_pos, retained, gaps)


def kv_cache_bytes(n_layers: int, n_kv_heads: int, head_dim: int, elem_bytes: int, seq_len: int) -> int:
    """KV-cache footprint, Eq. 2: 2 x layers x heads x dim_head x precision x sequence length."""
    return 2 * n_layers * n_kv_heads * head_dim * elem_bytes * seq_len
