// Tensor-core kernels for bf16 (sm_100a): attention (a1, Eq. 1) and score (a2, Eq. 4).
// Operands are staged in shared memory by TMA in the 128-byte-swizzled layouts tcgen05.mma reads,
// accumulators live in TMEM, and only the two dense contractions (Q K^T and P V) use the tensor
// cores; softmax, masking and the score reduction run on the CUDA cores in fp32.
#pragma once
#include <cuda.h>
#include "geom.cuh"
#include "ptx.cuh"

namespace kvc {

static constexpr int kSubTileBytes = 128 * 128;   // 128 rows x 64 bf16 (one 128-byte swizzled row each)

// Row packing shared by both kernels: for kv-head g the G query heads that share it are stacked
// with the tokens, row r = (token - tok0) * G + (head - g*G), so keys and values are read once per
// kv-head.  A tile holds TOK = 128 / G tokens (TOK * G <= 128 rows).


static constexpr int kStages = 4;                 // K/V ring slots of the attention kernel

// ------------------------------------------------------------------------------------------------
// a0 + a1: append (Alg. 1) and attention (Eq. 1).  Two 128-row tiles (A, B) per CTA, software pipelined,
// with the key range optionally split over the CTAs of a thread-block cluster.  Keys are the cache rows
// [0, n_c) followed by the block's own tokens, which are read from the k/v inputs directly.
//   warps 0-3   softmax of tile A     (thread = one row = one TMEM lane), 216 registers
//   warps 4-7   softmax of tile B
//   warp  8     TMA producer: Q tiles once, then K_j, V_j, K_j+1, ... through a ring of kStages 32 KB slots
//   warp  9     MMA issuer of tile A, warp 10 of tile B (one lane each).  Per key tile j an issuer
//               queues O_t += P_t V_j, then S_t = Q_t K_{j+1}^T.  P is handed over in two halves
//               (64 keys each) so the first PV MMAs start while the second half of the exponentials
//               is still being computed.  P -> P V -> next S -> softmax is the row tile's critical chain:
//               with two row tiles the next S is issued directly behind the second half of P V, and the
//               commits that free ring slots and publish O follow it.
//   warp  11    only gives its registers away (setmaxnreg works on groups of four warps)
// a0: the block's key / value tiles are stored into the cache from their ring slots (TMA stores issued by warp 9).
// The two softmax groups take turns on the exponentials (named barriers): while one tile's exponentials
// occupy the CUDA cores the tensor pipe runs the other tile's MMAs; without the hand-over both tiles fall
// into lockstep and the two pipes idle alternately.  Loading S and finding the maxima is outside the turn.
// (Measured and dropped: eight softmax warps per row tile, two threads per row, also in the form where a CTA
// with a single row tile lends it the other tile's warps -- no faster; a polynomial 2^x on the FMA pipe for part
// of the columns -- slower; S in two halves of 64 keys with the first issued early -- slower, MMAs with N = 64
// read Q twice as often; exponentials against the running maximum with the tile's maximum found afterwards --
// slower, the period is then bound by the two exponential phases, which that form lengthens.)
// TMEM columns: S_A/P_A [0,128)  S_B/P_B [128,256)  O_A [256,384)  O_B [384,512).
// The running output is rescaled lazily: a row keeps its reference maximum until the true maximum
// has grown by more than 2^8, so P stays below 256 and O rarely needs touching.
//
// Key split: with cluster size S the CTA of cluster rank s handles key tiles [s*T/S, (s+1)*T/S) of
// its row-tile pair and ends with a partial (O, m, l).  The partials are exchanged through
// distributed shared memory: rank s owns rows [s*128/S, (s+1)*128/S) of both tiles.  With two row tiles
// every CTA copies its partial rows (fp32) into the owner's shared memory with remote stores, the cluster
// synchronises, and each rank combines and writes its rows.  With one row tile the rows (with m and l
// behind them) leave in one bulk copy per owner, which completes on a barrier of the owner.  Nothing but
// the final result goes to HBM.
// Row tiles per CTA: R = 2 as described, or R = 1.  A CTA with one row tile runs it twice over: softmax group and
// issuer t take its key tiles t, t+2, ... with S, P, O, maximum and row sum of their own (tile B's TMEM columns), and
// the two partial results are merged at the end.  That costs about 1.1 times as much per row tile and key tile, but
// exchanges half as much in the combine and doubles the CTA count, which lets a launch that would need S = 4 do
// with S = 2; the host picks.
// grid (ceil(ceil(n/TOK)/R) * S, Hkv, nl), cluster (S,1,1), block 384,
// dynamic smem (2 + kStages) * (D/64) * 16 KB + 1 KB.
static constexpr int kAttnThreads = 384;

struct TcSmemAttn {
  uint64_t q_full[2], kv_full[kStages], kv_empty[kStages], s_full[2], p_half[2][2], pv_done[2];
  uint64_t comb_full;        // key split: the other ranks' partial rows have landed in this CTA's shared memory
  uint32_t tmem_base;
  int wait_ctl[2];           // [0] abort flag, [1] wait limit in units of 1024 cycles (see mbar_wait)
  alignas(16) float stat[2 * 128 * 2];   // (read and written as float2) key split: (m, l) of the rows this rank owns, [S sources][2 tiles][rows_per][2], S * rows_per = 128
};

template <int D>
__global__ void __launch_bounds__(kAttnThreads, 1) attn_tc_kernel(const __grid_constant__ CUtensorMap tm_q,
                                                                   const __grid_constant__ CUtensorMap tm_k,
                                                                   const __grid_constant__ CUtensorMap tm_v,
                                                                   const __grid_constant__ CUtensorMap tm_kin,
                                                                   const __grid_constant__ CUtensorMap tm_vin,
                                                                   char* __restrict__ cache,
                                                                   __nv_bfloat16* __restrict__ out,
                                                                   char* __restrict__ ws, Geom p, int S, int R) {
  constexpr int NSUB = D / 64;
  constexpr int TILE_BYTES = NSUB * kSubTileBytes;
  constexpr uint32_t TMEM_COLS = 512;
  constexpr float kRescaleThreshold = 8.f;      // log2 units
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sQ = smem;                            // two tiles
  uint8_t* ring = smem + 2 * TILE_BYTES;         // kStages tiles; after the key loop: the parked O tiles
  __shared__ TcSmemAttn sh;

  const int layer = blockIdx.z, g = blockIdx.y;
  const int split = S > 1 ? static_cast<int>(cluster_ctarank()) : 0;
  const int pair = blockIdx.x / S;               // index of this CTA's group of R row tiles (R = 1 or 2)
  const int TOK = 128 / p.G, rows = TOK * p.G;
  const int tokA = pair * R * TOK, tokB = tokA + TOK;
  const bool has_B = R == 2 && tokB < p.n;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int last_tok = min(tokA + R * TOK, p.n) - 1;
  // Key tiles this pair of row tiles can see: Tc tiles of the cache (rows [0, n_c), the last one possibly
  // partial), then the block's own keys in tiles of 128 tokens, read straight from the k/v inputs.
  const int Tc = (p.n_c + 127) / 128;
  const int T = Tc + (last_tok + 128) / 128;
  const int t_begin = split * T / S, t_end = (split + 1) * T / S;
  const int Tl = t_end - t_begin;                // key tiles of this CTA (0 is possible when S > T)
  // A CTA with one row tile and at least two key tiles runs the tile twice over: softmax group and issuer t take the
  // key tiles t, t+2, ... with accumulators, maxima and sums of their own (the TMEM columns of tile B are free), two
  // key tiles are in flight as with two row tiles, and the two partial results are merged at the end.
  const bool alt = !has_B && Tl >= 2;
  const int n_it[2] = {alt ? (Tl + 1) / 2 : Tl, alt ? Tl / 2 : (has_B ? Tl : 0)};   // key tiles of group 0 / 1

  if (threadIdx.x == 0) {
    for (int i = 0; i < 2; ++i) {
      mbar_init(&sh.q_full[i], 1); mbar_init(&sh.s_full[i], 1); mbar_init(&sh.pv_done[i], 1);
      mbar_init(&sh.p_half[i][0], 4); mbar_init(&sh.p_half[i][1], 4);     // one arrival per softmax warp
    }
    // a ring slot is free again once the issuer of every active row tile has committed its MMAs on it
    for (int i = 0; i < kStages; ++i) { mbar_init(&sh.kv_full[i], 1); mbar_init(&sh.kv_empty[i], has_B ? 2 : 1); }
    sh.wait_ctl[0] = 0; sh.wait_ctl[1] = p.wait_limit_k;
    mbar_init(&sh.comb_full, 1);
    // key split with one row tile: every other rank of the cluster will copy its partial of this rank's rows here
    if (S > 1 && !has_B) mbar_expect_tx(&sh.comb_full, (S - 1) * (128 / S) * (D + 4) * 4);
    mbar_fence_init();
  }
  // rows of the Q tiles that TMA never writes (rows >= TOK*G) must still be finite
  {
    const int pad16 = (128 - rows) * 8;          // 16-byte units per sub-tile
    for (int i = threadIdx.x; i < 2 * NSUB * pad16; i += blockDim.x) {
      const int sub = i / pad16, rem = i % pad16;
      reinterpret_cast<uint4*>(sQ + sub * kSubTileBytes + rows * 128)[rem] = make_uint4(0, 0, 0, 0);
    }
  }
  fence_proxy_async_smem();
  if (warp == 8) {
    tmem_alloc(&sh.tmem_base, TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = sh.tmem_base;
  volatile int* abort_flag = sh.wait_ctl;

  if (warp >= 8) {
    reg_dec<72>();
    if (warp == 8) {
      // ---------------------------------------------------------------- TMA producer
      if (lane == 0) {
        tma_prefetch_desc(&tm_q); tma_prefetch_desc(&tm_k); tma_prefetch_desc(&tm_v);
        tma_prefetch_desc(&tm_kin); tma_prefetch_desc(&tm_vin);
      }
      // While the previous kernel drains: ask L2 for the Q tiles and the first two key / value tiles (a hint only,
      // nothing is read into the SM before the wait below), so that the first loads find them there.
      if (Tl > 0 && lane < 2 + 2 * NSUB * min(Tl, 2)) {
        if (lane < 2) {
          if (lane == 0 || has_B)
            for (int sub = 0; sub < NSUB; ++sub) tma_prefetch_l2_4d(&tm_q, sub * 64, g * p.G, lane ? tokB : tokA, layer);
        } else {
          const int i = (lane - 2) / NSUB, sub = (lane - 2) % NSUB;      // ring item i: K or V of key tile t_begin + i/2
          const int kt = t_begin + (i >> 1);
          if (kt < Tc) tma_prefetch_l2_4d((i & 1) ? &tm_v : &tm_k, sub * 64, kt * 128, g, layer);
          else tma_prefetch_l2_4d((i & 1) ? &tm_vin : &tm_kin, sub * 64, g, (kt - Tc) * 128, layer);
        }
      }
      __syncwarp();
      if (lane == 0) {
        pdl_wait();                                // the block's keys were appended by the previous kernel
        stamp_begin(p);
      }
      if (lane == 0 && Tl > 0) {
        mbar_expect_tx(&sh.q_full[0], NSUB * rows * 128);
        for (int sub = 0; sub < NSUB; ++sub)
          tma_load_4d(sQ + sub * kSubTileBytes, &tm_q, &sh.q_full[0], sub * 64, g * p.G, tokA, layer);
        if (has_B) {
          mbar_expect_tx(&sh.q_full[1], NSUB * rows * 128);
          for (int sub = 0; sub < NSUB; ++sub)
            tma_load_4d(sQ + TILE_BYTES + sub * kSubTileBytes, &tm_q, &sh.q_full[1], sub * 64, g * p.G, tokB, layer);
        }
        for (int i = 0; i < 2 * Tl; ++i) {         // item 2j = K of tile t_begin + j, item 2j+1 = V of it
          const int slot = i % kStages, round = i / kStages;
          if (round > 0 && !mbar_wait(&sh.kv_empty[slot], (round - 1) & 1, abort_flag)) break;
          mbar_expect_tx(&sh.kv_full[slot], TILE_BYTES);
          const int kt = t_begin + (i >> 1);
          if (kt < Tc) {                           // cache rows kt*128 .. (rows past n_c are masked by the softmax)
            const CUtensorMap* tm = (i & 1) ? &tm_v : &tm_k;
            for (int sub = 0; sub < NSUB; ++sub)
              tma_load_4d(ring + slot * TILE_BYTES + sub * kSubTileBytes, tm, &sh.kv_full[slot], sub * 64, kt * 128, g, layer);
          } else {                                 // block tokens (kt - Tc)*128 .. (tokens past n are zero-filled)
            const CUtensorMap* tm = (i & 1) ? &tm_vin : &tm_kin;
            for (int sub = 0; sub < NSUB; ++sub)
              tma_load_4d(ring + slot * TILE_BYTES + sub * kSubTileBytes, tm, &sh.kv_full[slot], sub * 64, g, (kt - Tc) * 128, layer);
          }
        }
      }
    } else if (warp == 9 || (warp == 10 && (has_B || alt))) {
      // ---------------------------------------------------------------- MMA issuer of tile t
      // a0 append (Alg. 1: C <- C u (K_i, V_i)).  The block's keys and values pass through the ring as key tiles
      // anyway: the issuer of tile A stores such a tile from its ring slot into cache rows n_c + 128u .. with one
      // TMA store per 64 columns (rows past the block are zero in the tile and land in unused cache rows or are
      // clipped at cap).  Among the CTAs that load block tile u, the one whose rows contain token 128u owns it.
      // Nobody in this kernel reads the appended rows.  The lanes of the warp write the positions.
      const int u_lo = max(t_begin, Tc) - Tc, u_hi = t_end - Tc;            // block tiles of this CTA: [u_lo, u_hi)
      auto owns = [&](int u) { return (u * 128) / (R * TOK) == pair; };
      if (warp == 9 && u_hi > u_lo) {
        bool waited = false;
        for (int u = u_lo; u < u_hi; ++u) {
          if (!owns(u)) continue;
          if (!waited) { pdl_wait(); waited = true; }                       // the previous block's compaction is done with the cache
          int* pos = reinterpret_cast<int*>(cache + layer * p.cache_ls + p.pos_off) + static_cast<long long>(g) * p.cap + p.n_c;
          for (int i = u * 128 + lane; i < min(p.n, u * 128 + 128); i += 32) pos[i] = static_cast<int>(p.pos0 + i);
        }
      }
      if (lane == 0 && Tl > 0) {
        const int t = warp - 9;
        bool stored = false, store_waited = false;
        // item i of the ring (2j = K, 2j+1 = V of local key tile j) has landed in `slot`: store it if it is ours
        // (with two row tiles the issuer of tile A stores, else the issuer that consumes the item);
        // true if the slot must not be handed back before the store has read it
        auto append_item = [&](int i, int slot) {
          const int u = t_begin + (i >> 1) - Tc;
          if ((t != 0 && !alt) || u < 0 || !owns(u)) return false;
          if (!store_waited) { pdl_wait(); store_waited = true; }
          const CUtensorMap* tm = (i & 1) ? &tm_v : &tm_k;
          for (int sub = 0; sub < NSUB; ++sub)
            tma_store_4d(tm, ring + slot * TILE_BYTES + sub * kSubTileBytes, sub * 64, p.n_c + u * 128, g, layer);
          tma_store_commit();
          stored = true;
          return i + kStages < 2 * Tl;
        };
        constexpr uint32_t idesc_qk = idesc_bf16_f32(128, 128, 0, 0);
        constexpr uint32_t idesc_pv = idesc_bf16_f32(128, D, 0, 1);
        constexpr uint32_t hi = smem_desc_hi_sw128(1024);
        const uint32_t q_lo = smem_desc_lo(smem_u32(sQ) + (alt ? 0 : t) * TILE_BYTES, 16);   // K-major operand
        const uint32_t k_lo0 = smem_desc_lo(smem_u32(ring), 16);                        // K-major operand
        const uint32_t v_lo0 = smem_desc_lo(smem_u32(ring), kSubTileBytes);             // MN-major operand
        const uint32_t tS = tmem + t * 128, tO = tmem + 256 + t * 128;
        const int first = alt ? t : 0, step = alt ? 2 : 1;   // local key tiles of this issuer: first, first + step, ...
        auto issue_S = [&](int slot) {               // S_t = Q_t K^T, 16 of the d columns per MMA
          const uint32_t k_lo = k_lo0 + slot * (TILE_BYTES >> 4);
#pragma unroll
          for (int kk = 0; kk < D / 16; ++kk) {
            const uint32_t off = ((kk / 4) * kSubTileBytes + (kk % 4) * 32) >> 4;
            mma_ss_lh(tS, q_lo + off, hi, k_lo + off, hi, idesc_qk, kk > 0);
          }
        };
        auto issue_PV = [&](int slot, int half, bool acc) {   // O_t += P_t V, 16 keys per MMA, 64 keys per half
          const uint32_t v_lo = v_lo0 + slot * (TILE_BYTES >> 4);
#pragma unroll
          for (int kk = 4 * half; kk < 4 * half + 4; ++kk)
            mma_ts_lh(tO, tS + kk * 8, v_lo + kk * (2048 >> 4), hi, idesc_pv, acc || kk > 0);
        };
        const int i0 = 2 * first;                    // ring item of this issuer's first K tile (slot i0, first round)
        bool ok = mbar_wait(&sh.q_full[alt ? 0 : t], 0, abort_flag) && mbar_wait(&sh.kv_full[i0], 0, abort_flag);
        if (ok) {
          tc_fence_after_sync();
          issue_S(i0);
          mma_commit(&sh.s_full[t]);
          if (append_item(i0, i0)) tma_store_wait_read();
          mma_commit(&sh.kv_empty[i0]);
        }
        for (int jj = first, it = 0; jj < Tl && ok; jj += step, ++it) {
          const int jn = jj + step;                  // the key tile whose S is queued behind P V of this one
          const int iv = 2 * jj + 1, ik = 2 * jn;
          const int slotV = iv % kStages, slotK = ik % kStages;
          ok = mbar_wait_spin(&sh.p_half[t][0], it & 1, abort_flag) && mbar_wait(&sh.kv_full[slotV], (iv / kStages) & 1, abort_flag);
          if (!ok) break;
          tc_fence_after_sync();
          issue_PV(slotV, 0, it > 0);
          const bool hold_v = append_item(iv, slotV);
          // What follows the second half of P is the row tile's critical chain (P -> P V -> next S -> softmax).  With
          // two row tiles nothing else sits between the two groups of MMAs: the next K tile (landed long ago) is
          // waited for here, and the commits that free the slots and publish O come after the next S has been issued
          // (they then complete with it, which nobody minds: O is read after the next S at the earliest).  In-kernel
          // stamps put the commits and the wait at 380 of the chain's 4000 cycles.  With one row tile and two key
          // chains every ring item feeds one chain only and the ring holds one key tile per chain: there the V slot
          // goes back to the producer first, and the K tile is waited for when it is needed (measured: the deferred
          // order starves the other chain and costs 13 %).
          const bool defer = !alt;
          if (defer && jn < Tl) {
            ok = mbar_wait(&sh.kv_full[slotK], (ik / kStages) & 1, abort_flag);
            if (!ok) break;
          }
          ok = mbar_wait_spin(&sh.p_half[t][1], it & 1, abort_flag);
          if (!ok) break;
          tc_fence_after_sync();
          issue_PV(slotV, 1, true);
          if (!defer) {
            mma_commit(&sh.pv_done[t]);
            if (hold_v) tma_store_wait_read();
            mma_commit(&sh.kv_empty[slotV]);
            if (jn < Tl) {
              ok = mbar_wait(&sh.kv_full[slotK], (ik / kStages) & 1, abort_flag);
              if (!ok) break;
              tc_fence_after_sync();
            }
          }
          if (jn < Tl) {
            issue_S(slotK);
            mma_commit(&sh.s_full[t]);
          }
          if (defer) {
            mma_commit(&sh.pv_done[t]);
            if (hold_v) tma_store_wait_read();
            mma_commit(&sh.kv_empty[slotV]);
          }
          if (jn < Tl) {
            if (append_item(ik, slotK)) tma_store_wait_read();
            mma_commit(&sh.kv_empty[slotK]);
          }
        }
        // the stores have read their ring slots (the combine of a key split reuses the ring) ...
        if (stored) tma_store_wait_read();
      }
    }
    __syncwarp();
    // Key split with one row tile: softmax group 0 writes over the ring once both key chains are complete, which says
    // nothing about the stores above; warps 9 and 10 tell it here that no store reads the ring any more.
    if (S > 1 && !has_B && (warp == 9 || warp == 10)) named_barrier_arrive(6, 128 + 64);
    if (lane == 0) tma_store_wait_all();        // ... and the appended rows are in the cache before the kernel ends
    if (S > 1) {                                             // the cluster barriers of the combine below
      cluster_arrive(); cluster_wait();
      cluster_arrive(); cluster_wait();
    }
  } else {
    reg_inc<216>();
    // ---------------------------------------------------------------- softmax + epilogue of tile t
    const int t = warp >> 2;
    const int r = (warp & 3) * 32 + lane;                     // row of the tile = TMEM lane
    const int tok0 = (t && !alt) ? tokB : tokA;             // (both groups hold the rows of tile A when they alternate)
    const int tok = tok0 + r / p.G, hh = r % p.G;
    const bool row_valid = r < rows && tok < p.n;
    const uint32_t lane_addr = static_cast<uint32_t>((warp & 3) * 32) << 16;
    const uint32_t tmem_S = tmem + t * 128 + lane_addr, tmem_O = tmem + 256 + t * 128 + lane_addr;
    float m_ref = -INFINITY, l = 0.f;                        // reference maximum (log2 units) and row sum
    float wm0 = 1.f, wm1 = 0.f;                              // key split, one row tile: weights of the two key chains' O
    bool ok = true;
    const bool writer = t == 0 || has_B;                     // this group writes results (a row tile of its own)
    const bool active = writer || alt;                       // this group takes part in the key loop
    const int first = alt ? t : 0, step = alt ? 2 : 1;       // local key tiles of this group: first, first + step, ...
    // Turn taking (named barrier 2 + t = "group t may go", 128 waiters + 128 arrivals).  Group 0 goes first.
    const bool turns = (has_B || alt) && Tl > 0;
    if (turns && t == 1) named_barrier_arrive(2, 256);
    if (active) {
      for (int jj = first, it = 0; jj < Tl; jj += step, ++it) {
        const int kt = t_begin + jj;                          // key tile index
        // Waits that gave up only skip the arithmetic: the turn barrier is passed on every path, once per key
        // tile and warp, so the other row tile never waits for a turn that is not handed over.
        if (ok) ok = __all_sync(0xffffffffu, mbar_wait(&sh.s_full[t], it & 1, abort_flag));
        bool took_turn = false;
        if (ok) do {
        tc_fence_after_sync();
        uint32_t sr[128];
#pragma unroll
        for (int c = 0; c < 4; ++c) tmem_ld32(tmem_S + c * 32, sr + c * 32);
        tmem_wait_ld();
        // columns [0, lim) of this tile are visible: a cache tile ends at row n_c, a block tile at the row's
        // own token (causal inside the block); only the last cache tile and diagonal tiles need the mask
        const int u = kt - Tc;                                // >= 0: tile of the block's own tokens
        const int lim = u < 0 ? p.n_c - kt * 128 : tok + 1 - u * 128;
        if (u < 0 ? lim < 128 : (u + 1) * 128 > tok0 + 1) {
#pragma unroll
          for (int c = 0; c < 128; ++c)
            if (c >= lim) sr[c] = 0xff800000u;                // -inf
        }
        float mx4[8];                                         // independent chains of three-input maxima
#pragma unroll
        for (int i = 0; i < 8; ++i) mx4[i] = fmaxf(__uint_as_float(sr[i]), __uint_as_float(sr[8 + i]));
#pragma unroll
        for (int c = 16; c < 128; c += 16) {
#pragma unroll
          for (int i = 0; i < 8; ++i) mx4[i] = fmax3(mx4[i], __uint_as_float(sr[c + i]), __uint_as_float(sr[c + 8 + i]));
        }
        const float mx = fmaxf(fmax3(mx4[0], mx4[1], mx4[2]), fmaxf(fmax3(mx4[3], mx4[4], mx4[5]), fmaxf(mx4[6], mx4[7])));
        const float m_new = mx * p.scale_log2;                // scale > 0
        if (it == 0) {
          m_ref = m_new == -INFINITY ? 0.f : m_new;
        } else {
          const bool grow = m_new > m_ref + kRescaleThreshold;
          if (__any_sync(0xffffffffu, grow)) {
            const float f = grow ? fast_exp2(m_ref - m_new) : 1.f;
            if (grow) { m_ref = m_new; l *= f; }
            ok = __all_sync(0xffffffffu, mbar_wait(&sh.pv_done[t], (it - 1) & 1, abort_flag));  // O_t holds every earlier tile
            if (!ok) break;
            tc_fence_after_sync();
#pragma unroll
            for (int c = 0; c < D / 32; ++c) {
              uint32_t o[32];
              tmem_ld32(tmem_O + c * 32, o);
              tmem_wait_ld();
#pragma unroll
              for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * f);
              tmem_st32(tmem_O + c * 32, o);
            }
          }
        }
        // Only the exponentials are taken in turns: loading S and finding the row maxima overlap the other
        // tile's exponentials.
        if (turns) { named_barrier(2 + t, 256); took_turn = true; }
        // (packed fp32: one instruction scales two columns, one adds two exponentials to the partial sums)
        const uint64_t scale2 = f32x2(p.scale_log2, p.scale_log2), neg_m2 = f32x2(-m_ref, -m_ref);
        uint64_t ps2[2] = {f32x2(0.f, 0.f), f32x2(0.f, 0.f)};
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          uint32_t pk[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            float x0, x1;
            f32x2_split(fma_f32x2(f32x2(__uint_as_float(sr[c * 32 + 2 * i]), __uint_as_float(sr[c * 32 + 2 * i + 1])), scale2, neg_m2), x0, x1);
            const float p0 = fast_exp2(x0), p1 = fast_exp2(x1);
            ps2[i & 1] = add_f32x2(ps2[i & 1], f32x2(p0, p1));
            pk[i] = pack_bf16x2(p0, p1);
          }
          tmem_st16(tmem_S + c * 16, pk);
          if (c & 1) {                                        // 64 keys of P are in TMEM: release them to the MMA warp
            tmem_wait_st();
            tc_fence_before_sync();
            // one arrival per warp: 128 arrivals on one shared-memory word are served one after the other, and the
            // issuer saw the barrier complete some 300 cycles after the first of them (in-kernel stamps)
            __syncwarp();
            if (lane == 0) mbar_arrive(&sh.p_half[t][c >> 1]);
          }
        }
        {
          float ps[4];
          f32x2_split(ps2[0], ps[0], ps[1]);
          f32x2_split(ps2[1], ps[2], ps[3]);
          l += (ps[0] + ps[1]) + (ps[2] + ps[3]);
        }
        } while (0);
        if (turns && !took_turn) named_barrier(2 + t, 256);   // a wait gave up before the turn was taken: take it now
        // hand the turn over if the other group has a key tile left: its it-th (group 0 asks) or (it+1)-th (group 1)
        if (turns && (t == 0 ? it < n_it[1] : it + 1 < n_it[0])) named_barrier_arrive(3 - t, 256);
      }
      // The key loop is over: the next kernel of the stream may be scheduled and set itself up while this one
      // writes its results.  (Triggered at the start instead, the waiting CTAs of the next attention launch take the
      // SMs that the compress kernel of the previous layer, ready on a side stream, could use.)
      if (threadIdx.x == 0) pdl_launch_dependents();
      if (ok && n_it[t] > 0) ok = mbar_wait(&sh.pv_done[t], (n_it[t] - 1) & 1, abort_flag);
      ok = __all_sync(0xffffffffu, ok);                       // the TMEM accesses below are warp-wide
      if (ok && n_it[t] > 0) tc_fence_after_sync();
      if (alt && S == 1) {
        // Merge and write out, half the columns per group: group t keeps columns [t*D/2, (t+1)*D/2) of its O in
        // registers and parks the other half (fp32, 16-byte chunks XOR-swizzled with row & 7 against bank conflicts)
        // and its (m, l) in shared memory over the Q tiles, which nobody reads once both groups are past their
        // last P V; then each group combines its columns of both partial results and writes them.
        constexpr int H = D / 2;
        float* mrg = reinterpret_cast<float*>(smem);          // [2 groups][128][H]
        named_barrier(5, 256);
        if (ok) {
#pragma unroll
          for (int c = 0; c < H / 32; ++c) {
            uint32_t o[32];
            tmem_ld32(tmem_O + (1 - t) * H + c * 32, o);
            tmem_wait_ld();
#pragma unroll
            for (int k = 0; k < 8; ++k)
              *reinterpret_cast<uint4*>(mrg + (t * 128 + r) * H + (((c * 8 + k) ^ (r & 7)) << 2)) = make_uint4(o[4 * k], o[4 * k + 1], o[4 * k + 2], o[4 * k + 3]);
          }
        }
        sh.stat[(t * 128 + r) * 2] = (ok && l > 0.f) ? m_ref : -INFINITY;   // -inf: this group saw no key of the row
        sh.stat[(t * 128 + r) * 2 + 1] = l;
        named_barrier(5, 256);
        if (ok) {
          const float m1 = sh.stat[((1 - t) * 128 + r) * 2], l1 = sh.stat[((1 - t) * 128 + r) * 2 + 1];
          const float m0 = l > 0.f ? m_ref : -INFINITY;
          const float m_all = fmaxf(m0, m1);                   // finite: group 0 has seen key tile 0, hence a key of every row
          const float w0 = fast_exp2(m0 - m_all), w1 = fast_exp2(m1 - m_all);
          const float L = fmaf(w1, l1, w0 * l);
          const float inv = 1.f / L, a0 = w0 * inv, a1 = w1 * inv;
          __nv_bfloat16* orow = out + layer * p.out_ls + (static_cast<long long>(tok) * p.Hq + g * p.G + hh) * D + t * H;
#pragma unroll
          for (int c = 0; c < H / 32; ++c) {
            uint32_t o[32];
            tmem_ld32(tmem_O + t * H + c * 32, o);
            tmem_wait_ld();
            if (row_valid) {
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                const float4 b0 = *reinterpret_cast<const float4*>(mrg + ((1 - t) * 128 + r) * H + (((c * 8 + 2 * i) ^ (r & 7)) << 2));
                const float4 b1 = *reinterpret_cast<const float4*>(mrg + ((1 - t) * 128 + r) * H + (((c * 8 + 2 * i + 1) ^ (r & 7)) << 2));
                uint4 vv;
                vv.x = pack_bf16x2(fmaf(a1, b0.x, a0 * __uint_as_float(o[8 * i + 0])), fmaf(a1, b0.y, a0 * __uint_as_float(o[8 * i + 1])));
                vv.y = pack_bf16x2(fmaf(a1, b0.z, a0 * __uint_as_float(o[8 * i + 2])), fmaf(a1, b0.w, a0 * __uint_as_float(o[8 * i + 3])));
                vv.z = pack_bf16x2(fmaf(a1, b1.x, a0 * __uint_as_float(o[8 * i + 4])), fmaf(a1, b1.y, a0 * __uint_as_float(o[8 * i + 5])));
                vv.w = pack_bf16x2(fmaf(a1, b1.z, a0 * __uint_as_float(o[8 * i + 6])), fmaf(a1, b1.w, a0 * __uint_as_float(o[8 * i + 7])));
                reinterpret_cast<uint4*>(orow + c * 32)[i] = vv;
              }
            }
          }
          if (row_valid && t == 0) {
            float* lse = reinterpret_cast<float*>(ws_slot(ws, p, layer) + p.lse_off);
            lse[static_cast<long long>(tok) * p.Hq + g * p.G + hh] = (m_all + log2f(L)) * 0.6931471805599453f;
          }
        }
      } else if (alt) {
        // Key split: merge the two groups' partial results into group 0's accumulator for the cluster combine below: group 1 parks its rows of O (fp32, 16-byte
        // chunks XOR-swizzled with row & 7 against bank conflicts) and (m, l) in shared memory over the Q tiles, which
        // nobody reads once both groups are past their last P V; group 0 rescales both to the common maximum.
        float* mrg = reinterpret_cast<float*>(smem);          // [128][D]
        named_barrier(5, 256);
        if (t == 1) {
          if (ok) {
#pragma unroll
            for (int c = 0; c < D / 32; ++c) {
              uint32_t o[32];
              tmem_ld32(tmem_O + c * 32, o);
              tmem_wait_ld();
#pragma unroll
              for (int k = 0; k < 8; ++k)
                *reinterpret_cast<uint4*>(mrg + r * D + (((c * 8 + k) ^ (r & 7)) << 2)) = make_uint4(o[4 * k], o[4 * k + 1], o[4 * k + 2], o[4 * k + 3]);
            }
          }
          sh.stat[2 * r] = (ok && l > 0.f) ? m_ref : -INFINITY;   // -inf: this group saw no key of the row
          sh.stat[2 * r + 1] = l;
        }
        named_barrier(5, 256);
        if (t == 0 && ok) {
          // (a key split has one row tile here -- R = 1 -- or two; with one, the rows of chain 1 stay parked and are
          // folded in when group 0 stages its rows for the cluster: only m and l are merged now)
          const float m1 = sh.stat[2 * r], l1 = sh.stat[2 * r + 1];
          if (m1 != -INFINITY) {
            const float m_all = fmaxf(m_ref, m1);              // group 0 has seen key tile 0, hence a key of every row
            wm0 = fast_exp2(m_ref - m_all);
            wm1 = fast_exp2(m1 - m_all);
            l = fmaf(wm1, l1, wm0 * l);
            m_ref = m_all;
          }
        }
      }
      if (S == 1 && writer && !alt) {
        if (ok) {
          const float inv = 1.f / l;
          __nv_bfloat16* orow = out + layer * p.out_ls + (static_cast<long long>(tok) * p.Hq + g * p.G + hh) * D;
#pragma unroll
          for (int c = 0; c < D / 32; ++c) {
            uint32_t o[32];
            tmem_ld32(tmem_O + c * 32, o);
            tmem_wait_ld();
            if (row_valid) {
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                uint4 vv;
                vv.x = pack_bf16x2(__uint_as_float(o[8 * i + 0]) * inv, __uint_as_float(o[8 * i + 1]) * inv);
                vv.y = pack_bf16x2(__uint_as_float(o[8 * i + 2]) * inv, __uint_as_float(o[8 * i + 3]) * inv);
                vv.z = pack_bf16x2(__uint_as_float(o[8 * i + 4]) * inv, __uint_as_float(o[8 * i + 5]) * inv);
                vv.w = pack_bf16x2(__uint_as_float(o[8 * i + 6]) * inv, __uint_as_float(o[8 * i + 7]) * inv);
                reinterpret_cast<uint4*>(orow + c * 32)[i] = vv;
              }
            }
          }
          if (row_valid) {
            float* lse = reinterpret_cast<float*>(ws_slot(ws, p, layer) + p.lse_off);
            lse[static_cast<long long>(tok) * p.Hq + g * p.G + hh] = (m_ref + log2f(l)) * 0.6931471805599453f;
          }
        }
      }
    }
    if (S > 1 && !has_B) {
      // Combine the partials of the cluster, one row tile (S is a power of two; rank s owns rows [s*rows_per,
      // (s+1)*rows_per)).  Group 0 writes its rows of O -- the two key chains folded together with the weights found
      // above, chain 1 read from where group 1 parked it -- into a staging tile whose rows carry (m, l) behind the D
      // values; the rows of every other owner then leave in ONE bulk copy each (shared memory to the owner's shared
      // memory, completing on a barrier of the owner: this GPU's memory, no multicast), and each rank reduces its rows
      // from the staging tile (its own partial) and from what the others sent:
      //   O = sum_s 2^(m_s - m*) O_s / sum_s 2^(m_s - m*) l_s.
      // Shared memory: the parked rows [128][D] over the Q tiles; over the ring the received rows [S - 1 sources]
      // [rows_per][D + 4] and the staging tile [128][D + 4] (a row stride of D + 4 floats keeps thread-per-row
      // accesses off each other's banks).
      constexpr int RS = D + 4;
      const int rows_per = 128 / S;
      const float* mrg = reinterpret_cast<const float*>(smem);
      float* recv = reinterpret_cast<float*>(smem + 2 * TILE_BYTES);
      float* stg = recv + (128 - rows_per) * RS;
      // This CTA's own ring is free: both key chains are complete, the producer loads no tile that is not used, and
      // the issuer warps arrive on barrier 6 once the stores of the appended tiles have read their slots.
      if (t == 0) {
        named_barrier(6, 128 + 64);
        const bool have = ok && Tl > 0;                         // warp-uniform
#pragma unroll
        for (int c = 0; c < D / 32; ++c) {
          uint32_t o[32];
          if (have) {
            tmem_ld32(tmem_O + c * 32, o);
            tmem_wait_ld();
          } else {
#pragma unroll
            for (int i = 0; i < 32; ++i) o[i] = 0u;
          }
#pragma unroll
          for (int k = 0; k < 8; ++k) {
            float4 v4 = make_float4(__uint_as_float(o[4 * k]), __uint_as_float(o[4 * k + 1]), __uint_as_float(o[4 * k + 2]), __uint_as_float(o[4 * k + 3]));
            if (have && alt && wm1 != 0.f) {                  // (0: chain 1 saw no key of the row, or gave up)
              const float4 b4 = *reinterpret_cast<const float4*>(mrg + r * D + (((c * 8 + k) ^ (r & 7)) << 2));
              v4.x = fmaf(wm1, b4.x, wm0 * v4.x); v4.y = fmaf(wm1, b4.y, wm0 * v4.y);
              v4.z = fmaf(wm1, b4.z, wm0 * v4.z); v4.w = fmaf(wm1, b4.w, wm0 * v4.w);
            }
            *reinterpret_cast<float4*>(stg + r * RS + (c * 8 + k) * 4) = v4;
          }
        }
        *reinterpret_cast<float4*>(stg + r * RS + D) = make_float4((have && l > 0.f) ? m_ref : -INFINITY, have ? l : 0.f, 0.f, 0.f);
        fence_proxy_async_smem();                               // the rows just written are read by bulk copies
      }
      // Every CTA of the cluster has staged its rows and is done with its ring, where the copies land.  (The barrier
      // also orders this rank's staged rows before the reads of group 1 below.)
      cluster_arrive();
      cluster_wait();
      if (threadIdx.x == 0) {
        for (int owner = 0; owner < S; ++owner) {
          if (owner == split) continue;
          const int slot = split < owner ? split : split - 1;   // this rank among the owner's other ranks
          bulk_copy_to_cluster(dsmem_addr(smem_u32(recv + slot * rows_per * RS), owner), smem_u32(stg + owner * rows_per * RS),
                               rows_per * RS * 4, dsmem_addr(smem_u32(&sh.comb_full), owner));
        }
      }
      ok = mbar_wait(&sh.comb_full, 0, abort_flag) && ok;       // the other ranks' rows have landed
      {
        const int r0 = split * rows_per;
        const int per_tile = rows_per * (D / 32);               // work items: (row, group of 32 columns)
        for (int item = threadIdx.x; item < per_tile; item += 256) {
          const int lr = item % rows_per, cg = item / rows_per, r = r0 + lr;
          const int tok = tokA + r / p.G, hh = r % p.G;
          if (!(r < rows && tok < p.n)) continue;
          auto row_of = [&](int s2) -> const float* {
            return s2 == split ? stg + r * RS : recv + ((s2 < split ? s2 : s2 - 1) * rows_per + lr) * RS;
          };
          float m_all = -INFINITY;
#pragma unroll 1
          for (int s2 = 0; s2 < S; ++s2) m_all = fmaxf(m_all, row_of(s2)[D]);
          float L = 0.f;
          float acc[32];
#pragma unroll
          for (int i = 0; i < 32; ++i) acc[i] = 0.f;
#pragma unroll 1
          for (int s2 = 0; s2 < S; ++s2) {
            const float* row = row_of(s2);
            const float2 ml = *reinterpret_cast<const float2*>(row + D);
            if (ml.x == -INFINITY) continue;                  // this source saw no key of the row
            const float wt = fast_exp2(ml.x - m_all);
            L = fmaf(wt, ml.y, L);
#pragma unroll
            for (int k = 0; k < 8; ++k) {
              const float4 v4 = *reinterpret_cast<const float4*>(row + (cg * 8 + k) * 4);
              acc[4 * k + 0] = fmaf(wt, v4.x, acc[4 * k + 0]);
              acc[4 * k + 1] = fmaf(wt, v4.y, acc[4 * k + 1]);
              acc[4 * k + 2] = fmaf(wt, v4.z, acc[4 * k + 2]);
              acc[4 * k + 3] = fmaf(wt, v4.w, acc[4 * k + 3]);
            }
          }
          const float inv = 1.f / L;
          __nv_bfloat16* orow = out + layer * p.out_ls + (static_cast<long long>(tok) * p.Hq + g * p.G + hh) * D + cg * 32;
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            uint4 vv;
            vv.x = pack_bf16x2(acc[8 * i + 0] * inv, acc[8 * i + 1] * inv);
            vv.y = pack_bf16x2(acc[8 * i + 2] * inv, acc[8 * i + 3] * inv);
            vv.z = pack_bf16x2(acc[8 * i + 4] * inv, acc[8 * i + 5] * inv);
            vv.w = pack_bf16x2(acc[8 * i + 6] * inv, acc[8 * i + 7] * inv);
            reinterpret_cast<uint4*>(orow)[i] = vv;
          }
          if (cg == 0) {
            float* lse = reinterpret_cast<float*>(ws_slot(ws, p, layer) + p.lse_off);
            lse[static_cast<long long>(tok) * p.Hq + g * p.G + hh] = (m_all + log2f(L)) * 0.6931471805599453f;
          }
        }
      }
      // A CTA must not exit while a bulk copy still reads its staging tile: every rank has waited for the copies
      // addressed to it, so once all of them are here every copy is complete.
      cluster_arrive();
      cluster_wait();
    } else if (S > 1) {
      // Combine the partials of the cluster, two row tiles (S is a power of two).  Rank s owns rows [s*rows_per, (s+1)*rows_per)
      // of both tiles.  Tile by tile, the softmax threads park their rows of O (fp32: the output tolerance
      // leaves no room for a 16-bit exchange format) in a local staging tile, then copy it row by row into
      // the owners' shared memory with remote stores -- stores are not waited for, remote loads would be --
      // so that every warp instruction writes 512 contiguous bytes (one 16-byte store per thread straight
      // from the TMEM layout, thread = row, scatters 32 rows per instruction and moved 13 B/clk).  The
      // cluster synchronises, and each rank reduces its rows from its own shared memory:
      //   O = sum_s 2^(m_s - m*) O_s / sum_s 2^(m_s - m*) l_s.
      // recv: [S sources][2 tiles][rows_per][D] fp32 over the Q tiles and the first half of the ring; staging
      // [128][D] behind it; the 16-byte chunks of a row are XOR-swizzled with (row & 7) so that neither the
      // writers (lane = row) nor the readers (lane = row, same chunk) collide on banks.
      const int rows_per = 128 / S;
      float* stage = reinterpret_cast<float*>(smem);            // recv
      float* stg = stage + 2 * 128 * D;
      float* stat = sh.stat;                                    // [S][2][rows_per][2]: m (-inf: row saw no key), l
      cluster_arrive();                                         // every CTA is done with its Q tiles and ring
      cluster_wait();
      {
        constexpr int nthr = 256;                               // both groups take part
        const bool have = ok && Tl > 0;                         // warp-uniform
        for (int tt = 0; tt < 2; ++tt) {
          if (t == tt) {
            const int owner = r / rows_per, lr = r - owner * rows_per;
#pragma unroll
            for (int c = 0; c < D / 32; ++c) {
              uint32_t o[32];
              if (have) {
                tmem_ld32(tmem_O + c * 32, o);
                tmem_wait_ld();
              } else {
#pragma unroll
                for (int i = 0; i < 32; ++i) o[i] = 0u;
              }
#pragma unroll
              for (int k = 0; k < 8; ++k)
                *reinterpret_cast<uint4*>(stg + r * D + (((c * 8 + k) ^ (lr & 7)) << 2)) = make_uint4(o[4 * k], o[4 * k + 1], o[4 * k + 2], o[4 * k + 3]);
            }
            uint32_t stat_addr = smem_u32(stat + ((split * 2 + tt) * rows_per + lr) * 2);
            if (owner != split) stat_addr = dsmem_addr(stat_addr, owner);
            dsmem_st_v2(stat_addr, (have && l > 0.f) ? m_ref : -INFINITY, have ? l : 0.f);
          }
          named_barrier(1, nthr);                               // the staging tile is complete
          constexpr int CPR = D / 4;                            // 16-byte chunks per row
#pragma unroll 4
          for (int idx = threadIdx.x; idx < 128 * CPR; idx += nthr) {
            const int row = idx / CPR, chunk = idx % CPR;
            const int owner = row / rows_per, lr = row - owner * rows_per;
            const uint4 v4 = *reinterpret_cast<const uint4*>(stg + row * D + chunk * 4);
            uint32_t dst = smem_u32(stage + ((split * 2 + tt) * rows_per + lr) * D + chunk * 4);
            if (owner != split) dst = dsmem_addr(dst, owner);
            dsmem_st_v4_b32(dst, v4.x, v4.y, v4.z, v4.w);
          }
          named_barrier(1, nthr);                               // the staging tile may be overwritten
        }
      }
      cluster_arrive();                                         // all partials have landed; no remote access is
      cluster_wait();                                           // started after this
      {
        const int r0 = min(128, split * rows_per), nrows = min(128, r0 + rows_per) - r0;
        const int per_tile = nrows * (D / 32);                  // work items: (row, group of 32 columns)
        for (int item = threadIdx.x; item < 2 * per_tile; item += 256) {
          const int t = item / per_tile, rem = item % per_tile;
          const int lr = rem % nrows, cg = rem / nrows, r = r0 + lr;
          const int tok = (t ? tokB : tokA) + r / p.G, hh = r % p.G;
          if (!(r < rows && tok < p.n)) continue;
          // (the loops over the sources are kept rolled: this code runs once per CTA, straight-line copies of it
          // cost more in instruction fetch than the loop does in branches)
          float m_all = -INFINITY;
#pragma unroll 1
          for (int s = 0; s < S; ++s) m_all = fmaxf(m_all, stat[((s * 2 + t) * rows_per + lr) * 2]);
          float L = 0.f;
          float acc[32];
#pragma unroll
          for (int i = 0; i < 32; ++i) acc[i] = 0.f;
#pragma unroll 1
          for (int s = 0; s < S; ++s) {
            const float2 ml = *reinterpret_cast<const float2*>(stat + ((s * 2 + t) * rows_per + lr) * 2);
            if (ml.x == -INFINITY) continue;                  // this source saw no key of the row
            const float wt = fast_exp2(ml.x - m_all);
            L = fmaf(wt, ml.y, L);
            const float* row = stage + ((s * 2 + t) * rows_per + lr) * D;
#pragma unroll
            for (int k = 0; k < 8; ++k) {
              const float4 v4 = *reinterpret_cast<const float4*>(row + (((cg * 8 + k) ^ (lr & 7)) << 2));
              acc[4 * k + 0] = fmaf(wt, v4.x, acc[4 * k + 0]);
              acc[4 * k + 1] = fmaf(wt, v4.y, acc[4 * k + 1]);
              acc[4 * k + 2] = fmaf(wt, v4.z, acc[4 * k + 2]);
              acc[4 * k + 3] = fmaf(wt, v4.w, acc[4 * k + 3]);
            }
          }
          const float inv = 1.f / L;
          __nv_bfloat16* orow = out + layer * p.out_ls + (static_cast<long long>(tok) * p.Hq + g * p.G + hh) * D + cg * 32;
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            uint4 vv;
            vv.x = pack_bf16x2(acc[8 * i + 0] * inv, acc[8 * i + 1] * inv);
            vv.y = pack_bf16x2(acc[8 * i + 2] * inv, acc[8 * i + 3] * inv);
            vv.z = pack_bf16x2(acc[8 * i + 4] * inv, acc[8 * i + 5] * inv);
            vv.w = pack_bf16x2(acc[8 * i + 6] * inv, acc[8 * i + 7] * inv);
            reinterpret_cast<uint4*>(orow)[i] = vv;
          }
          if (cg == 0) {
            float* lse = reinterpret_cast<float*>(ws_slot(ws, p, layer) + p.lse_off);
            lse[static_cast<long long>(tok) * p.Hq + g * p.G + hh] = (m_all + log2f(L)) * 0.6931471805599453f;
          }
        }
      }
    }
  }

  tc_fence_before_sync();
  __syncthreads();
  if (warp == 8) {
    tc_fence_after_sync();
    tmem_dealloc(tmem, TMEM_COLS);
  }
  if (threadIdx.x == 0) stamp_end(p);
  if (threadIdx.x == 0 && sh.wait_ctl[0]) atomicExch(reinterpret_cast<int*>(ws), -4 /* KVC_ETIMEOUT */);
}

// ------------------------------------------------------------------------------------------------
// a2 score: one CTA per 128 candidate keys of one kv-head.  S^T = K_tile Q_obs^T puts keys on the
// TMEM lanes, so each thread owns one key and sums 2^(s*scale_log2 - lse2) over the observer
// columns in its own registers.  Observer rows are processed in groups of up to 256 columns.
// grid (ceil(n_cand/128), Hkv, nl), block 128, dynamic smem (D/64)*16 KB + (D/64)*32 KB + 1 KB.
struct TcSmemScore {
  uint64_t bar_k, bar_q, bar_s;
  uint32_t tmem_base;
  int wait_ctl[2];           // [0] abort flag, [1] wait limit in units of 1024 cycles (see mbar_wait)
  alignas(16) float lse2[256];
};

template <int D>
__global__ void __launch_bounds__(128) score_tc_kernel(const __grid_constant__ CUtensorMap tm_k,
                                                       const __grid_constant__ CUtensorMap tm_qobs,
                                                       char* __restrict__ ws, Geom p, int tok_per_group) {
  constexpr int NSUB = D / 64;
  constexpr uint32_t TMEM_COLS = 256;
  constexpr int kQSubBytes = 256 * 128;        // up to 256 observer rows x 128 B
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sK = smem;
  uint8_t* sQ = sK + NSUB * kSubTileBytes;
  __shared__ TcSmemScore sh;

  const int layer = blockIdx.z, g = blockIdx.y, key0 = blockIdx.x * 128;
  const int warp = threadIdx.x >> 5;
  char* slot = ws_slot(ws, p, layer);
  const float* lse = reinterpret_cast<const float*>(slot + p.lse_off);
  float* score = reinterpret_cast<float*>(slot + p.score_off) + static_cast<long long>(g) * p.cap;

  if (threadIdx.x == 0) {
    stamp_begin(p);
    mbar_init(&sh.bar_k, 1); mbar_init(&sh.bar_q, 1); mbar_init(&sh.bar_s, 1);
    sh.wait_ctl[0] = 0; sh.wait_ctl[1] = p.wait_limit_k;
    mbar_fence_init();
  }
  // observer rows beyond the last group's real rows are padding: keep them finite
  for (int i = threadIdx.x; i < NSUB * kQSubBytes / 16; i += blockDim.x)
    reinterpret_cast<uint4*>(sQ)[i] = make_uint4(0, 0, 0, 0);
  fence_proxy_async_smem();
  if (warp == 0) {
    tmem_alloc(&sh.tmem_base, TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = sh.tmem_base;
  volatile int* abort_flag = sh.wait_ctl;
  const uint32_t lane_addr = static_cast<uint32_t>(warp * 32) << 16;

  if (threadIdx.x == 0) {
    tma_prefetch_desc(&tm_k); tma_prefetch_desc(&tm_qobs);
    mbar_expect_tx(&sh.bar_k, NSUB * kSubTileBytes);
    for (int sub = 0; sub < NSUB; ++sub)
      tma_load_4d(sK + sub * kSubTileBytes, &tm_k, &sh.bar_k, sub * 64, key0, g, layer);
  }
  float acc = 0.f;
  bool ok = true;
  const int n_groups = (p.w + tok_per_group - 1) / tok_per_group;
  for (int grp = 0; grp < n_groups && ok; ++grp) {
    const int t_first = p.n - p.w + grp * tok_per_group;               // first observer token of the group
    const int t_cnt = min(tok_per_group, p.n - t_first);
    const int cols = t_cnt * p.G;                                      // real observer columns
    const int n_mma = (cols + 15) & ~15;                               // MMA N: multiple of 16, <= 256
    // everyone is past the previous group's TMEM reads and smem reads
    tc_fence_before_sync();
    __syncthreads();
    for (int c = threadIdx.x; c < 256; c += blockDim.x) {
      float lv = INFINITY;                                             // padding column: 2^-inf = 0
      if (c < cols) lv = lse[static_cast<long long>(t_first + c / p.G) * p.Hq + g * p.G + c % p.G] * 1.4426950408889634f;
      sh.lse2[c] = lv;
    }
    if (threadIdx.x == 0) {
      // the box always spans tok_per_group tokens; tokens past n are zero-filled by TMA
      mbar_expect_tx(&sh.bar_q, NSUB * tok_per_group * p.G * 128);
      for (int sub = 0; sub < NSUB; ++sub)
        tma_load_4d(sQ + sub * kQSubBytes, &tm_qobs, &sh.bar_q, sub * 64, g * p.G, t_first, layer);
      if (grp == 0) ok = mbar_wait(&sh.bar_k, 0, abort_flag);
      ok = ok && mbar_wait(&sh.bar_q, grp & 1, abort_flag);
      if (ok) {
        tc_fence_after_sync();
        const uint32_t idesc = idesc_bf16_f32(128, n_mma, 0, 0);
        const uint32_t aK = smem_u32(sK), aQ = smem_u32(sQ);
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk)
          mma_ss(tmem, smem_desc_sw128(aK + (kk / 4) * kSubTileBytes + (kk % 4) * 32, 16, 1024),
                 smem_desc_sw128(aQ + (kk / 4) * kQSubBytes + (kk % 4) * 32, 16, 1024), idesc, kk > 0);
        mma_commit(&sh.bar_s);
      }
    }
    __syncwarp();
    __syncthreads();                                                   // lse2 visible
    ok = mbar_wait(&sh.bar_s, grp & 1, abort_flag);
    if (!ok) break;
    tc_fence_after_sync();
    for (int c0 = 0; c0 < n_mma; c0 += 16) {
      uint32_t sr[16];
      tmem_ld16(tmem + lane_addr + c0, sr);
      tmem_wait_ld();
#pragma unroll
      for (int i = 0; i < 16; ++i) acc += fast_exp2(__uint_as_float(sr[i]) * p.scale_log2 - sh.lse2[c0 + i]);
    }
  }
  const int key = key0 + threadIdx.x;
  if (ok && key < p.n_cand) score[key] = acc;
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after_sync();
    tmem_dealloc(tmem, TMEM_COLS);
  }
  if (threadIdx.x == 0) stamp_end(p);
  if (threadIdx.x == 0 && sh.wait_ctl[0]) atomicExch(reinterpret_cast<int*>(ws), -4 /* KVC_ETIMEOUT */);
}

}  // namespace kvc
