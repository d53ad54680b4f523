// a2 + a3 + a4 in one launch: importance scores (Eq. 4), exact selection of the entries to evict
// (Alg. 1, Evict) and hole-fill compaction back to the budget M (the last step of Alg. 1's loop body).
//
// One thread-block cluster of Cn CTAs per (kv-head, layer).
//   phase 1 (MODE = kScoreAttention, bf16)  the 128-key tiles of the candidates are dealt round-robin to the CTAs
//            of the cluster.  Per tile: K tile by TMA, S^T = K_tile Q_obs^T on the tensor cores (keys on
//            the TMEM lanes, observer rows on the columns), each thread sums 2^(s*scale - lse2) over
//            the observer columns of its key and writes the score.  Two tiles are in flight per CTA
//            (two K buffers, two TMEM accumulators, two epilogue warp groups).
//            MODE = kScoresGiven: the scores are already in the workspace (score kernel of its own).
//            MODE = kScoreKeyDiff: query-agnostic score 1 - cos(k_j, mean key) (Sec. 3.2), any dtype.
//   phase 2  cluster barrier; then EVERY CTA reads all scores of its kv-head (L2-resident), builds the
//            64-bit keys in shared memory and runs the same exact selection redundantly -- cheaper than
//            a distributed histogram, since the SM-to-SM path is narrow and the other SMs would idle.
//   phase 3  every CTA derives the same ordered hole / survivor lists and executes every Cn-th move.
// Entry j gets the key (score bits << 32) | ~pos: a larger key means a higher score and, at equal
// score, an older entry; keys are unique because positions are.  Scores are sums of probabilities,
// hence >= 0, so their IEEE bit patterns order like integers.  The n_keep-th largest key (the cut-off)
// is found exactly by an MSB-first radix descent with 11-bit digits that starts below the bits all
// keys share and stops as soon as the bin that holds the cut-off survives as a whole.
#pragma once
#include <cuda.h>
#include <type_traits>
#include "geom.cuh"
#include "ptx.cuh"

namespace kvc {

// 512 threads and at most ~108 KB of shared memory per CTA: two CTAs share an SM, so that one scores
// (TMA / tensor-core bound) while the other selects (barrier bound) when many kv-heads are in flight.
static constexpr int kCompressThreads = 512;
static constexpr int kDigitBits = 11;
static constexpr int kSelBins = 1 << kDigitBits;
static constexpr int kRankMax = 256;          // keys of the cut-off bin that are ranked directly instead of by further rounds
static constexpr int kMaxKeysSmem = 6144;     // candidates whose keys fit the shared-memory table (48 KB)
static constexpr int kMaxMovesSmem = 2048;    // moves whose (src, dst) fit the shared-memory tables (16 KB)
static constexpr int kMaxObsRowsFused = 128;  // observer rows (w * G) the fused scoring phase takes
static constexpr int kMaxClusterWide = 16;   // largest cluster the host asks for (non-portable size: more than 8 CTAs)
static constexpr int kScoresGiven = 0, kScoreAttention = 1, kScoreKeyDiff = 2;   // what phase 1 of compress_kernel does
static constexpr int kSubTileBytesC = 128 * 128;

__device__ __forceinline__ unsigned long long select_key(float score, int pos) {
  return (static_cast<unsigned long long>(__float_as_uint(score)) << 32) |
         static_cast<unsigned long long>(0xFFFFFFFFu - static_cast<uint32_t>(pos));
}

// The selection and the listing run on the whole block (measured: a quarter of it pays less per barrier but more
// per key, and loses).
static constexpr int kTeam = kCompressThreads;

struct CompressSmem {
  uint64_t q_full, k_full[2], s_full[2], t_free[2];
  uint32_t tmem_base;
  int wait_ctl[2];           // [0] abort flag, [1] wait limit in units of 1024 cycles (see mbar_wait)
  alignas(16) float lse2[256];
  unsigned long long list[2 * (kTeam / 32) + 2];
  int scan_scratch[kTeam / 32 + 1];
  unsigned long long s_prefix;
  int s_remaining, s_bin_count, s_count;
};

// grid (Cn, Hkv, nl), cluster (Cn,1,1), block 512.
// dynamic smem: the larger of the scoring buffers (two K tiles + up to 128 observer rows) and of the key
// and move tables with the two histograms (80 KB), + 1 KB.
template <int D, int MODE>
__global__ void __launch_bounds__(kCompressThreads, 2) compress_kernel(const __grid_constant__ CUtensorMap tm_k,
                                                                       const __grid_constant__ CUtensorMap tm_qobs,
                                                                       char* __restrict__ cache, char* __restrict__ ws,
                                                                       Geom p, int Cn, int elem_bytes) {
  constexpr int NSUB = D / 64;
  constexpr int K_TILE_BYTES = NSUB * kSubTileBytesC;
  constexpr int kQSubBytes = kMaxObsRowsFused * 128;   // up to 128 observer rows x 128 B
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  __shared__ CompressSmem sh;

  const int layer = blockIdx.z, g = blockIdx.y;
  const int rank = Cn > 1 ? static_cast<int>(cluster_ctarank()) : 0;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  char* blob = cache + layer * p.cache_ls;
  int* pos = reinterpret_cast<int*>(blob + p.pos_off) + static_cast<long long>(g) * p.cap;
  char* slot = ws_slot(ws, p, layer);
  float* score = reinterpret_cast<float*>(slot + p.score_off) + static_cast<long long>(g) * p.cap;
  int* msrc_g = reinterpret_cast<int*>(slot + p.msrc_off) + static_cast<long long>(g) * p.max_chunk;
  int* mdst_g = reinterpret_cast<int*>(slot + p.mdst_off) + static_cast<long long>(g) * p.max_chunk;
  int* mcount = reinterpret_cast<int*>(slot + p.mcount_off);
  volatile int* abort_flag = sh.wait_ctl;
  if (tid == 0) { sh.wait_ctl[0] = 0; sh.wait_ctl[1] = p.wait_limit_k; }
  pdl_launch_dependents();                        // the next kernel of the stream may set itself up meanwhile

  // ------------------------------------------------------------------------------------ phase 1: scores
  if constexpr (MODE == kScoreAttention) {
    uint8_t* sK = smem;                              // two K tiles
    uint8_t* sQ = smem + 2 * K_TILE_BYTES;           // observer rows
    const int n_tiles = (p.n_cand + 127) / 128;
    const int my_tiles = rank < n_tiles ? (n_tiles - rank + Cn - 1) / Cn : 0;
    const int cols = p.w * p.G;                      // observer columns (<= 128: one MMA, two accumulators of 128 columns)
    const int n_mma = (cols + 15) & ~15;
    if (tid == 0) {
      mbar_init(&sh.q_full, 1);
      for (int i = 0; i < 2; ++i) { mbar_init(&sh.k_full[i], 1); mbar_init(&sh.s_full[i], 1); mbar_init(&sh.t_free[i], 4); }
      mbar_fence_init();
    }
    // observer rows beyond the real ones are padding: keep them finite
    for (int i = tid; i < NSUB * kQSubBytes / 16; i += kCompressThreads) reinterpret_cast<uint4*>(sQ)[i] = make_uint4(0, 0, 0, 0);
    fence_proxy_async_smem();
    if (warp == 8) {
      tmem_alloc(&sh.tmem_base, 256);
      tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = sh.tmem_base;
    if (warp == 8) {
      if (lane == 0) {
        tma_prefetch_desc(&tm_k); tma_prefetch_desc(&tm_qobs);
        pdl_wait();
        stamp_begin(p);
        bool ok = true;
        if (my_tiles > 0) {
          mbar_expect_tx(&sh.q_full, NSUB * p.w * p.G * 128);
          for (int sub = 0; sub < NSUB; ++sub)
            tma_load_4d(sQ + sub * kQSubBytes, &tm_qobs, &sh.q_full, sub * 64, g * p.G, p.n - p.w, layer);
          for (int i = 0; i < my_tiles && i < 2; ++i) {
            mbar_expect_tx(&sh.k_full[i], K_TILE_BYTES);
            for (int sub = 0; sub < NSUB; ++sub)
              tma_load_4d(sK + i * K_TILE_BYTES + sub * kSubTileBytesC, &tm_k, &sh.k_full[i], sub * 64,
                          (rank + i * Cn) * 128, g, layer);
          }
          ok = mbar_wait(&sh.q_full, 0, abort_flag);
        }
        const uint32_t idesc = idesc_bf16_f32(128, n_mma, 0, 0);
        constexpr uint32_t hi = smem_desc_hi_sw128(1024);
        const uint32_t k_lo0 = smem_desc_lo(smem_u32(sK), 16), q_lo = smem_desc_lo(smem_u32(sQ), 16);
        for (int i = 0; i < my_tiles && ok; ++i) {
          const int b = i & 1;
          ok = mbar_wait(&sh.k_full[b], (i >> 1) & 1, abort_flag);
          if (ok && i >= 2) ok = mbar_wait(&sh.t_free[b], ((i - 2) >> 1) & 1, abort_flag);   // accumulator b read out
          if (!ok) break;
          tc_fence_after_sync();
#pragma unroll
          for (int kk = 0; kk < D / 16; ++kk)
            mma_ss_lh(tmem + b * 128, k_lo0 + ((b * K_TILE_BYTES + (kk / 4) * kSubTileBytesC + (kk % 4) * 32) >> 4), hi,
                      q_lo + (((kk / 4) * kQSubBytes + (kk % 4) * 32) >> 4), hi, idesc, kk > 0);
          mma_commit(&sh.s_full[b]);
          if (i + 2 < my_tiles) {                    // refill K buffer b once the MMAs that read it are done
            ok = mbar_wait(&sh.s_full[b], (i >> 1) & 1, abort_flag);
            if (!ok) break;
            mbar_expect_tx(&sh.k_full[b], K_TILE_BYTES);
            for (int sub = 0; sub < NSUB; ++sub)
              tma_load_4d(sK + b * K_TILE_BYTES + sub * kSubTileBytesC, &tm_k, &sh.k_full[b], sub * 64,
                          (rank + (i + 2) * Cn) * 128, g, layer);
          }
        }
      }
      __syncwarp();
    } else if (warp < 8) {
      const int b = warp >> 2;
      const uint32_t lane_addr = static_cast<uint32_t>((warp & 3) * 32) << 16;
      pdl_wait();
      const float* lse = reinterpret_cast<const float*>(slot + p.lse_off);
      // log-sum-exp of the observer rows in log2 units; padding columns get +inf (2^-inf = 0).
      // Each epilogue group fills the whole table (same values), so no cross-group barrier is needed.
      for (int c = (warp & 3) * 32 + lane; c < 256; c += 128) {
        float lv = INFINITY;
        if (c < cols) lv = lse[static_cast<long long>(p.n - p.w + c / p.G) * p.Hq + g * p.G + c % p.G] * 1.4426950408889634f;
        sh.lse2[c] = lv;
      }
      named_barrier(1 + b, 128);
      bool ok = true;
      for (int i = b; i < my_tiles; i += 2) {
        ok = __all_sync(0xffffffffu, mbar_wait(&sh.s_full[b], (i >> 1) & 1, abort_flag));
        if (!ok) break;
        tc_fence_after_sync();
        float acc = 0.f;
        float acc2 = 0.f;
        for (int c0 = 0; c0 < n_mma; c0 += 32) {       // n_mma is a multiple of 16: the second half may be absent
          uint32_t sr[32];
          const bool two = c0 + 16 < n_mma;
          tmem_ld16(tmem + b * 128 + lane_addr + c0, sr);
          if (two) tmem_ld16(tmem + b * 128 + lane_addr + c0 + 16, sr + 16);
          tmem_wait_ld();
#pragma unroll
          for (int k = 0; k < 16; ++k) acc += fast_exp2(fmaf(__uint_as_float(sr[k]), p.scale_log2, -sh.lse2[c0 + k]));
          if (two) {
#pragma unroll
            for (int k = 16; k < 32; ++k) acc2 += fast_exp2(fmaf(__uint_as_float(sr[k]), p.scale_log2, -sh.lse2[c0 + k]));
          }
        }
        acc += acc2;
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh.t_free[b]);              // one arrival per warp of the epilogue group
        const int key = (rank + i * Cn) * 128 + (warp & 3) * 32 + lane;
        if (key < p.n_cand) score[key] = acc;
      }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 8) {
      tc_fence_after_sync();
      tmem_dealloc(tmem, 256);
    }
  } else if constexpr (MODE == kScoreKeyDiff) {
    // Query-agnostic score (Sec. 3.2): anchor mu = mean of the tot keys the cache holds after the append,
    // score_j = max(0, 1 - cos(k_j, mu)) for the candidates (>= 0, so its bit pattern orders like an integer; a
    // zero key or anchor has cosine 0).  A row is read by lpr lanes of 16 bytes; the CTAs of the cluster
    // take the 128-row tiles round-robin, add their partial sums through distributed shared memory, and
    // every CTA scores its own tiles (second read of K: L2).
    float* s_part = reinterpret_cast<float*>(smem);                 // [16 warps][d] partial sums
    float* s_sum = s_part + (kCompressThreads / 32) * 128;         // [d] this CTA's sum (read by the cluster)
    float* s_mu = s_sum + 128;                                      // [d] the anchor, [d] = its norm
    pdl_wait();
    if (tid == 0) stamp_begin(p);
    const int d = p.d, epl = 16 / elem_bytes;                       // elements per 16-byte piece: 8 (bf16) or 4 (fp32)
    const int lpr = d / epl, rpw = 32 / lpr;                        // lanes per row, rows per warp and step
    const int sub = lane / lpr, piece = lane % lpr;
    const long long row_bytes = static_cast<long long>(d) * elem_bytes;
    const char* Kg = blob + static_cast<long long>(g) * p.cap * row_bytes + piece * 16;
    auto fetch = [&](int row) { return *reinterpret_cast<const uint4*>(Kg + row * row_bytes); };
    auto widen = [&](const uint4 raw, float* f) {
      if (elem_bytes == 2) {
        const uint32_t w4[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) { f[2 * i] = __uint_as_float(w4[i] << 16); f[2 * i + 1] = __uint_as_float(w4[i] & 0xffff0000u); }
      } else {
        f[0] = __uint_as_float(raw.x); f[1] = __uint_as_float(raw.y); f[2] = __uint_as_float(raw.z); f[3] = __uint_as_float(raw.w);
#pragma unroll
        for (int i = 4; i < 8; ++i) f[i] = 0.f;
      }
    };
    const int tiles_all = (p.tot + 127) / 128;
    float acc[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[e] = 0.f;
    constexpr int kRowsInFlight = 4;                               // independent loads per lane: the pass is latency-bound otherwise
    const int rstep = (kCompressThreads / 32) * rpw;               // rows the CTA covers per step
    for (int tile = rank; tile < tiles_all; tile += Cn) {
      const int r_end = min(p.tot, tile * 128 + 128);
      for (int row = tile * 128 + warp * rpw + sub; row < r_end; row += rstep * kRowsInFlight) {
        uint4 raw[kRowsInFlight];
#pragma unroll
        for (int u = 0; u < kRowsInFlight; ++u)
          if (row + u * rstep < r_end) raw[u] = fetch(row + u * rstep);
#pragma unroll
        for (int u = 0; u < kRowsInFlight; ++u) {
          if (row + u * rstep < r_end) {
            float f[8];
            widen(raw[u], f);
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[e] += f[e];
          }
        }
      }
    }
    for (int o = lpr; o < 32; o <<= 1) {
#pragma unroll
      for (int e = 0; e < 8; ++e) acc[e] += __shfl_xor_sync(0xffffffffu, acc[e], o);
    }
    if (sub == 0)
      for (int e = 0; e < epl; ++e) s_part[warp * 128 + piece * epl + e] = acc[e];
    __syncthreads();
    if (tid < d) {
      float t = 0.f;
      for (int w2 = 0; w2 < kCompressThreads / 32; ++w2) t += s_part[w2 * 128 + tid];
      s_sum[tid] = t;
    }
    __syncthreads();
    if (Cn > 1) { cluster_arrive(); cluster_wait(); }
    if (tid < d) {
      float t = 0.f;
      if (Cn > 1) {
        const uint32_t a = smem_u32(&s_sum[tid]);
        for (int rk = 0; rk < Cn; ++rk) t += dsmem_ld_f32(dsmem_addr(a, rk));
      } else {
        t = s_sum[tid];
      }
      s_mu[tid] = t / static_cast<float>(p.tot);
    }
    __syncthreads();
    if (warp == 0) {
      float q2 = 0.f;
      for (int i = lane; i < d; i += 32) q2 += s_mu[i] * s_mu[i];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) q2 += __shfl_xor_sync(0xffffffffu, q2, o);
      if (lane == 0) s_mu[d] = sqrtf(q2);
    }
    __syncthreads();
    float mu[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) mu[e] = e < epl ? s_mu[piece * epl + e] : 0.f;
    const float mu_norm = s_mu[d];
    for (int tile = rank; tile < tiles_all; tile += Cn) {
      const int r_end = min(p.n_cand, tile * 128 + 128);
      for (int row0 = tile * 128 + warp * rpw; row0 < r_end; row0 += rstep * kRowsInFlight) {   // warp-uniform bound
        uint4 raw[kRowsInFlight];
#pragma unroll
        for (int u = 0; u < kRowsInFlight; ++u)
          if (row0 + sub + u * rstep < r_end) raw[u] = fetch(row0 + sub + u * rstep);
#pragma unroll
        for (int u = 0; u < kRowsInFlight; ++u) {
          const int row = row0 + sub + u * rstep;
          float dot = 0.f, nrm = 0.f;
          if (row < r_end) {
            float f[8];
            widen(raw[u], f);
#pragma unroll
            for (int e = 0; e < 8; ++e) { dot = fmaf(f[e], mu[e], dot); nrm = fmaf(f[e], f[e], nrm); }
          }
          for (int o = 1; o < lpr; o <<= 1) {
            dot += __shfl_xor_sync(0xffffffffu, dot, o);
            nrm += __shfl_xor_sync(0xffffffffu, nrm, o);
          }
          if (row < r_end && piece == 0) {
            // fp32 rounding can put the cosine of a key (nearly) parallel to the anchor a little above 1: clamp, so
            // that the score stays >= 0 and select_key's ordering by bit pattern holds
            const float den = sqrtf(nrm) * mu_norm;
            score[row] = den > 0.f ? fmaxf(0.f, 1.f - dot / den) : 1.f;
          }
        }
      }
    }
    __syncthreads();
  } else {
    if (tid == 0) { pdl_wait(); stamp_begin(p); }
    __syncthreads();
  }
  if (Cn > 1) {                                       // every score of this kv-head is in the workspace
    cluster_arrive();
    cluster_wait();
  } else {
    __syncthreads();
  }

  // ------------------------------------------------------------------------------------ phase 2: selection
  unsigned long long* keys = reinterpret_cast<unsigned long long*>(smem);           // 48 KB
  int* tab_src = reinterpret_cast<int*>(smem + kMaxKeysSmem * 8);                    // 8 KB
  int* tab_dst = tab_src + kMaxMovesSmem;                                            // 8 KB
  // histograms of two consecutive rounds (the second doubles as the list of the last bin's keys): 2 x 8 KB
  int (*hists)[kSelBins] = reinterpret_cast<int (*)[kSelBins]>(smem + kMaxKeysSmem * 8 + 2 * kMaxMovesSmem * 4);
  const bool keys_in_smem = p.n_cand <= kMaxKeysSmem;
  // One pass builds the keys (twelve independent loads in flight per thread: the scores come from L2), folds the
  // AND and the OR of all keys -- the bits above the highest bit in which any two keys differ are common to all of
  // them (scores of similar magnitude share their exponent bits), and the descent starts below them, so that the
  // first digit already spreads the keys over many bins -- and clears the first histogram.
  unsigned long long k_and = ~0ull, k_or = 0ull;
  constexpr int kKeyLoads = 12;                                  // independent (score, position) loads in flight per thread
  for (int j0 = tid; j0 < p.n_cand; j0 += kKeyLoads * kCompressThreads) {
    float sc[kKeyLoads];
    int ps[kKeyLoads];
#pragma unroll
    for (int u = 0; u < kKeyLoads; ++u) {
      const int j = j0 + u * kCompressThreads;
      if (j < p.n_cand) { sc[u] = __ldcg(score + j); ps[u] = pos[j]; }
    }
#pragma unroll
    for (int u = 0; u < kKeyLoads; ++u) {
      const int j = j0 + u * kCompressThreads;
      if (j < p.n_cand) {
        const unsigned long long k = select_key(sc[u], ps[u]);
        if (keys_in_smem) keys[j] = k;
        k_and &= k; k_or |= k;
      }
    }
  }
  {
    const unsigned a_lo = __reduce_and_sync(0xffffffffu, static_cast<unsigned>(k_and)), a_hi = __reduce_and_sync(0xffffffffu, static_cast<unsigned>(k_and >> 32));
    const unsigned o_lo = __reduce_or_sync(0xffffffffu, static_cast<unsigned>(k_or)), o_hi = __reduce_or_sync(0xffffffffu, static_cast<unsigned>(k_or >> 32));
    if (lane == 0) { sh.list[warp] = (static_cast<unsigned long long>(a_hi) << 32) | a_lo; sh.list[kTeam / 32 + warp] = (static_cast<unsigned long long>(o_hi) << 32) | o_lo; }
  }
  for (int i = tid; i < kSelBins; i += kTeam) hists[0][i] = 0;
  __syncthreads();
  // Selection and listing exist twice, for keys in shared memory and for keys re-read from the workspace: with the
  // choice made per access the compiler issues the global loads of the second form in both cases.
  const int n_lo = min(p.B, p.tot);
  const int max_moves = min(p.n, p.tot - p.B);                   // at most this many entries sit at or above row B
  const bool tabs_in_smem = max_moves <= kMaxMovesSmem;
  int* msrc = tabs_in_smem ? tab_src : msrc_g;                   // with global tables every CTA writes all entries
  int* mdst = tabs_in_smem ? tab_dst : mdst_g;                   // itself (same values) and reads only its own writes
  auto select_and_list = [&](auto in_smem) {
  constexpr bool kInSmem = decltype(in_smem)::value;
  auto key_of = [&](int j) -> unsigned long long {
    if constexpr (kInSmem) return keys[j];
    else return select_key(__ldcg(score + j), pos[j]);
  };
  unsigned long long thr = ~0ull;                                // n_keep == 0: nothing among the candidates survives
  if (p.n_keep > 0) {
    k_and = ~0ull; k_or = 0ull;
#pragma unroll
    for (int w2 = 0; w2 < kTeam / 32; ++w2) { k_and &= sh.list[w2]; k_or |= sh.list[kTeam / 32 + w2]; }   // (every thread: the same values)
    const unsigned long long differ = k_and ^ k_or;             // != 0: at least two distinct keys (n_cand > n_keep >= 1)
    const int top = 63 - __clzll(static_cast<long long>(differ));
    int shift = top >= kDigitBits - 1 ? top - (kDigitBits - 1) : 0, bits = top - shift + 1;
    // state of the descent, the same in every thread: the bits decided so far and the rank (1-based, from the top) of
    // the cut-off among the keys that share them
    unsigned long long prefix = top == 63 ? 0ull : (k_or >> (top + 1)) << (top + 1);
    int remaining = p.n_keep, hb = 0;
    while (true) {
      int* hist = hists[hb];
      const int hi = shift + bits;           // bits [hi, 64) are already decided
      for (int j = tid; j < p.n_cand; j += kTeam) {
        const unsigned long long key = key_of(j);
        if (hi >= 64 || (key >> hi) == (prefix >> hi)) atomicAdd(&hist[(key >> shift) & ((1u << bits) - 1)], 1);
      }
      for (int i = tid; i < kSelBins; i += kTeam) hists[hb ^ 1][i] = 0;   // for the next round
      __syncthreads();
      // descending scan: thread t owns the BPT bins from kSelBins - 1 - BPT*t downwards; scan inside the warp by
      // shuffles, across the warps by reading the totals of the warps before (one barrier)
      constexpr int BPT = kSelBins / kTeam;
      const int b0 = kSelBins - 1 - BPT * tid;
      int mine = 0;
#pragma unroll
      for (int i = 0; i < BPT; ++i) mine += hist[b0 - i];
      int incl = mine;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int y = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += y;
      }
      if (lane == 31) sh.scan_scratch[warp] = incl;
      __syncthreads();
      for (int w2 = 0; w2 < warp; ++w2) incl += sh.scan_scratch[w2];
      int excl = incl - mine;
      if (excl < remaining && remaining <= incl) {               // the cut-off lies in one of my bins
        int b = b0, h = hist[b0];
        while (excl + h < remaining) { excl += h; --b; h = hist[b]; }
        sh.s_prefix = prefix | (static_cast<unsigned long long>(b) << shift);
        sh.s_remaining = remaining - excl;                       // rank inside the chosen bin, 1-based
        sh.s_bin_count = h;
        sh.s_count = 0;
      }
      __syncthreads();
      prefix = sh.s_prefix; remaining = sh.s_remaining;
      const int h = sh.s_bin_count;
      // Done when every bit is decided, or when the whole bin survives (its rank equals its size): then
      // the prefix with zeros below it separates the retained keys from the others.
      if (shift == 0 || remaining == h) { thr = prefix; break; }
      if (h <= kRankMax) {
        // few keys left in the cut-off bin: list them and rank them directly (keys are unique: exactly one of them
        // has `remaining - 1` larger ones) instead of descending further
        unsigned long long* lst = reinterpret_cast<unsigned long long*>(hists[hb ^ 1]);
        for (int j = tid; j < p.n_cand; j += kTeam) {
          const unsigned long long key = key_of(j);
          if ((key >> shift) == (prefix >> shift)) lst[atomicAdd(&sh.s_count, 1)] = key;
        }
        __syncthreads();
        if (tid < h) {
          const unsigned long long my = lst[tid];
          int larger = 0;
          for (int i = 0; i < h; ++i) larger += lst[i] > my;
          if (larger == remaining - 1) sh.s_prefix = my;
        }
        __syncthreads();
        thr = sh.s_prefix;
        break;
      }
      bits = shift >= kDigitBits ? kDigitBits : shift;
      shift -= bits;
      hb ^= 1;
    }
  }

  // ------------------------------------------------------------------------------------ phase 3: compaction
  // holes: evicted entries in rows [0, B); survivors: retained entries in rows [B, tot), both in ascending
  // row order.  Entry j is retained iff it is protected (j >= n_cand) or its key >= thr.
  {
    // Every thread owns a run of consecutive rows: it counts its holes (rows below B) and survivors (rows from B
    // on), one scan over the block (shuffles inside the warps, one barrier across them) turns the counts into
    // offsets, and a second walk over the same rows writes the row indices, in ascending order.
    const int rpt = (p.tot + kTeam - 1) / kTeam;                 // rows per thread
    const int r0 = min(tid * rpt, p.tot), r1 = min(r0 + rpt, p.tot);
    auto retained = [&](int j) { return j >= p.n_cand || key_of(j) >= thr; };
    unsigned long long mine = 0;                                  // holes in the low word, survivors in the high word
    for (int j = r0; j < r1; ++j) {
      const bool keep = retained(j);
      if (j < n_lo) mine += keep ? 0ull : 1ull;
      else mine += keep ? (1ull << 32) : 0ull;
    }
    unsigned long long incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned long long y = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += y;
    }
    if (lane == 31) sh.list[warp] = incl;
    __syncthreads();
    unsigned long long before = 0, all = 0;
    for (int w2 = 0; w2 < kTeam / 32; ++w2) {
      const unsigned long long tw = sh.list[w2];
      if (w2 < warp) before += tw;
      all += tw;
    }
    const unsigned long long excl = before + incl - mine;
    int off_h = static_cast<int>(excl & 0xffffffffu), off_s = static_cast<int>(excl >> 32);
    const int total_holes = static_cast<int>(all & 0xffffffffu);
    for (int j = r0; j < r1; ++j) {
      const bool keep = retained(j);
      if (j < n_lo) { if (!keep) mdst[off_h++] = j; }
      else if (keep) msrc[off_s++] = j;
    }
    if (tid == 0) sh.s_remaining = total_holes;                  // == number of survivors: the cache returns to B
  }
  };
  if (keys_in_smem) select_and_list(std::true_type{}); else select_and_list(std::false_type{});
  __syncthreads();
  const int total_holes = sh.s_remaining;
  if (rank == 0 && tid == 0) mcount[g] = total_holes;
  if (Cn > 1) {                                                  // the moves overwrite positions (and rows) that the
    cluster_arrive();                                            // other CTAs of the cluster read while selecting
    cluster_wait();
  }

  // move m copies the K row, the V row and the position of entry src[m] (>= B) into the hole dst[m] (< B).
  // Sources and destinations never overlap, rows are copied bit-exactly.  One warp per move.
  const long long row_bytes = static_cast<long long>(p.d) * elem_bytes;
  const int vec = static_cast<int>(row_bytes / 16);
  const long long head = static_cast<long long>(g) * p.cap;
  // (row = 2 * vec pieces of 16 bytes, K then V; a warp keeps kMovesInFlight moves in flight, since one
  // load-then-store at a time would leave the copy latency-bound)
  constexpr int kMovesInFlight = 4;
  const int wstride = Cn * (kCompressThreads / 32);
  for (int mv0 = rank * (kCompressThreads / 32) + warp; mv0 < total_holes; mv0 += wstride * kMovesInFlight) {
    int src[kMovesInFlight], dst[kMovesInFlight];
#pragma unroll
    for (int u = 0; u < kMovesInFlight; ++u) {
      const int mv = mv0 + u * wstride;
      src[u] = mv < total_holes ? msrc[mv] : -1;
      dst[u] = mv < total_holes ? mdst[mv] : -1;
    }
    for (int i = lane; i < 2 * vec; i += 32) {
      const long long off = (i < vec ? 0 : p.v_off) + static_cast<long long>(i < vec ? i : i - vec) * 16;
      uint4 val[kMovesInFlight];
#pragma unroll
      for (int u = 0; u < kMovesInFlight; ++u)
        if (src[u] >= 0) val[u] = *reinterpret_cast<const uint4*>(blob + off + (head + src[u]) * row_bytes);
#pragma unroll
      for (int u = 0; u < kMovesInFlight; ++u)
        if (src[u] >= 0) *reinterpret_cast<uint4*>(blob + off + (head + dst[u]) * row_bytes) = val[u];
    }
    if (lane < kMovesInFlight && src[0] >= 0) {
      int sj = -1, dj = -1;
#pragma unroll
      for (int u = 0; u < kMovesInFlight; ++u)
        if (lane == u) { sj = src[u]; dj = dst[u]; }
      if (sj >= 0) pos[dj] = pos[sj];
    }
  }
  __syncthreads();
  if (tid == 0) stamp_end(p);
  if (tid == 0 && sh.wait_ctl[0]) atomicExch(reinterpret_cast<int*>(ws), -4 /* KVC_ETIMEOUT */);
}

}  // namespace kvc
