// CUDA-core kernels: append (a0), fp32-accurate attention (a1) and score (a2) for fp32 inputs
// (and, as a diagnostic, bf16 inputs).
#pragma once
#include "geom.cuh"
#include "ptx.cuh"

namespace kvc {

// ------------------------------------------------------------------------------------------------
// a0 append (Alg. 1: C <- C u (K_i, V_i)).  One warp per (token, kv-head) row: copies the K and V
// rows into cache rows n_c + t and records the absolute position.
// grid (ceil(n*Hkv / 8), 1, nl), block 256.
template <typename T>
__global__ void __launch_bounds__(256) append_kernel(const T* __restrict__ k, const T* __restrict__ v,
                                                     char* __restrict__ cache, Geom p) {
  pdl_launch_dependents();                 // the attention kernel may set itself up meanwhile
  pdl_wait();                              // the previous block's compaction still reads and writes this cache
  if (threadIdx.x == 0) stamp_begin(p);
  const int layer = blockIdx.z;
  const int row = blockIdx.x * 8 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (row < p.n * p.Hkv) {
    const int t = row / p.Hkv, g = row % p.Hkv;
    char* blob = cache + layer * p.cache_ls;
    const int vec_per_row = p.d * (int)sizeof(T) / 16;
    const uint4* ksrc = reinterpret_cast<const uint4*>(k + layer * p.kv_ls + (static_cast<long long>(t) * p.Hkv + g) * p.d);
    const uint4* vsrc = reinterpret_cast<const uint4*>(v + layer * p.kv_ls + (static_cast<long long>(t) * p.Hkv + g) * p.d);
    const long long dst_row = static_cast<long long>(g) * p.cap + p.n_c + t;
    uint4* kdst = reinterpret_cast<uint4*>(blob + dst_row * p.d * sizeof(T));
    uint4* vdst = reinterpret_cast<uint4*>(blob + p.v_off + dst_row * p.d * sizeof(T));
    for (int i = lane; i < vec_per_row; i += 32) {
      kdst[i] = ksrc[i];
      vdst[i] = vsrc[i];
    }
    if (lane == 0) reinterpret_cast<int*>(blob + p.pos_off)[dst_row] = static_cast<int>(p.pos0 + t);
  }
  __syncthreads();
  if (threadIdx.x == 0) stamp_end(p);
}

// ------------------------------------------------------------------------------------------------
// a1 attention on CUDA cores (Eq. 1), fp32 arithmetic throughout.
// Block = 4 warps x 4 rows = 16 tokens of one query head; keys/values stream through shared memory
// 32 at a time.  In the score phase lane j owns key j of the tile; in the PV phase lane c owns
// output columns c, c+32, ....  grid (ceil(n/16), Hq, nl), block 128.
template <typename T, int D>
__global__ void __launch_bounds__(128) attn_cc_kernel(const T* __restrict__ q, const char* __restrict__ cache,
                                                      T* __restrict__ out, char* __restrict__ ws, Geom p) {
  constexpr int RW = 4, KT = 32, KS = D + 4, NC = D / 32;
  __shared__ __align__(16) float sK[KT * KS];
  __shared__ __align__(16) float sV[KT * D];
  __shared__ __align__(16) float sQ[16 * D];
  if (threadIdx.x == 0) stamp_begin(p);
  const int layer = blockIdx.z, h = blockIdx.y, g = h / p.G;
  const int tok0 = blockIdx.x * 16;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const char* blob = cache + layer * p.cache_ls;
  const T* Kc = reinterpret_cast<const T*>(blob) + static_cast<long long>(g) * p.cap * D;
  const T* Vc = reinterpret_cast<const T*>(blob + p.v_off) + static_cast<long long>(g) * p.cap * D;
  const T* qb = q + layer * p.q_ls;

  for (int i = threadIdx.x; i < 16 * D; i += 128) {
    const int r = i / D, c = i % D, tok = tok0 + r;
    sQ[i] = tok < p.n ? to_f32<T>(qb[(static_cast<long long>(tok) * p.Hq + h) * D + c]) : 0.f;
  }

  float m[RW], l[RW], acc[RW][NC];
#pragma unroll
  for (int r = 0; r < RW; ++r) {
    m[r] = -INFINITY; l[r] = 0.f;
#pragma unroll
    for (int c = 0; c < NC; ++c) acc[r][c] = 0.f;
  }
  const int last_tok = min(tok0 + 16, p.n) - 1;
  const int kv_end = p.n_c + last_tok + 1;          // keys visible to the last row of this block

  for (int t0 = 0; t0 < kv_end; t0 += KT) {
    __syncthreads();
    for (int i = threadIdx.x; i < KT * D; i += 128) {
      const int j = i / D, c = i % D, key = t0 + j;
      float kk = 0.f, vv = 0.f;
      if (key < kv_end) {
        kk = to_f32<T>(Kc[static_cast<long long>(key) * D + c]);
        vv = to_f32<T>(Vc[static_cast<long long>(key) * D + c]);
      }
      sK[j * KS + c] = kk;
      sV[j * D + c] = vv;
    }
    __syncthreads();

    float s[RW];
#pragma unroll
    for (int r = 0; r < RW; ++r) s[r] = 0.f;
    const float4* krow = reinterpret_cast<const float4*>(&sK[lane * KS]);
#pragma unroll 8
    for (int c4 = 0; c4 < D / 4; ++c4) {
      const float4 kv = krow[c4];
#pragma unroll
      for (int r = 0; r < RW; ++r) {
        const float4 qv = reinterpret_cast<const float4*>(&sQ[(warp * RW + r) * D])[c4];
        s[r] = fmaf(qv.x, kv.x, s[r]); s[r] = fmaf(qv.y, kv.y, s[r]);
        s[r] = fmaf(qv.z, kv.z, s[r]); s[r] = fmaf(qv.w, kv.w, s[r]);
      }
    }
    const int key = t0 + lane;
    float pr[RW];
#pragma unroll
    for (int r = 0; r < RW; ++r) {
      const int tok = tok0 + warp * RW + r;
      const bool vis = tok < p.n && key < p.n_c + tok + 1;     // causal inside the block only
      const float t = vis ? s[r] * p.scale_log2 : -INFINITY;
      float tmax = t;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, o));
      const float m_new = fmaxf(m[r], tmax);
      float pv = 0.f, corr = 1.f;
      if (m_new != -INFINITY) {
        pv = exp2f(t - m_new);
        corr = exp2f(m[r] - m_new);
      }
      float psum = pv;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) psum += __shfl_xor_sync(0xffffffffu, psum, o);
      l[r] = l[r] * corr + psum;
      m[r] = m_new;
#pragma unroll
      for (int c = 0; c < NC; ++c) acc[r][c] *= corr;
      pr[r] = pv;
    }
#pragma unroll 4
    for (int j = 0; j < KT; ++j) {
      float vj[NC];
#pragma unroll
      for (int c = 0; c < NC; ++c) vj[c] = sV[j * D + lane + 32 * c];
#pragma unroll
      for (int r = 0; r < RW; ++r) {
        const float pj = __shfl_sync(0xffffffffu, pr[r], j);
#pragma unroll
        for (int c = 0; c < NC; ++c) acc[r][c] = fmaf(pj, vj[c], acc[r][c]);
      }
    }
  }

  float* lse = reinterpret_cast<float*>(ws_slot(ws, p, layer) + p.lse_off);
  T* ob = out + layer * p.out_ls;
#pragma unroll
  for (int r = 0; r < RW; ++r) {
    const int tok = tok0 + warp * RW + r;
    if (tok >= p.n) continue;
    const float inv = 1.f / l[r];
#pragma unroll
    for (int c = 0; c < NC; ++c)
      ob[(static_cast<long long>(tok) * p.Hq + h) * D + lane + 32 * c] = from_f32<T>(acc[r][c] * inv);
    if (lane == 0) lse[static_cast<long long>(tok) * p.Hq + h] = (m[r] + log2f(l[r])) * 0.6931471805599453f;
  }
  __syncthreads();
  if (threadIdx.x == 0) stamp_end(p);
}

// ------------------------------------------------------------------------------------------------
// a2 score on CUDA cores (Eq. 4): score_j = sum over the w observer rows and the G heads of the
// group of 2^(s_ij*scale_log2 - lse2_i).  A CTA owns 8 candidate keys; sixteen threads share a key and
// split the observer rows between them (the sum over rows is the long serial chain otherwise, and a launch
// of this path has a few hundred keys at most: many small CTAs, not few long ones).
// grid (ceil(n_cand/8), Hkv, nl), block 128, dynamic smem = 8*(D+4)*4 + 32*D*4 + 32*4 bytes.
static constexpr int kScoreCcKeys = 8;

template <typename T, int D>
__global__ void __launch_bounds__(128) score_cc_kernel(const T* __restrict__ q, const char* __restrict__ cache,
                                                       char* __restrict__ ws, Geom p) {
  constexpr int KS = D + 4;
  extern __shared__ __align__(16) float smem_f[];
  float* sK = smem_f;                          // [32][KS]
  float* sQ = sK + kScoreCcKeys * KS;          // [32][D]
  float* sL = sQ + 32 * D;                     // [32]
  if (threadIdx.x == 0) stamp_begin(p);
  const int layer = blockIdx.z, g = blockIdx.y;
  const int key0 = blockIdx.x * kScoreCcKeys;
  const char* blob = cache + layer * p.cache_ls;
  const T* Kc = reinterpret_cast<const T*>(blob) + static_cast<long long>(g) * p.cap * D;
  const T* qb = q + layer * p.q_ls;
  char* slot = ws_slot(ws, p, layer);
  const float* lse = reinterpret_cast<const float*>(slot + p.lse_off);
  float* score = reinterpret_cast<float*>(slot + p.score_off) + static_cast<long long>(g) * p.cap;

  for (int i = threadIdx.x; i < kScoreCcKeys * D; i += 128) {
    const int j = i / D, c = i % D, key = key0 + j;
    sK[j * KS + c] = key < p.n_cand ? to_f32<T>(Kc[static_cast<long long>(key) * D + c]) : 0.f;
  }
  const int rows = p.w * p.G;
  const int kj = threadIdx.x >> 4, part = threadIdx.x & 15;     // key of the CTA, sixteenth of the observer rows
  float acc = 0.f;
  const float4* krow = reinterpret_cast<const float4*>(&sK[kj * KS]);
  for (int r0 = 0; r0 < rows; r0 += 32) {
    __syncthreads();
    for (int i = threadIdx.x; i < 32 * D; i += 128) {
      const int r = r0 + i / D, c = i % D;
      float x = 0.f;
      if (r < rows) {
        const int tok = p.n - p.w + r / p.G, h = g * p.G + r % p.G;
        x = to_f32<T>(qb[(static_cast<long long>(tok) * p.Hq + h) * D + c]);
      }
      sQ[i] = x;
    }
    if (threadIdx.x < 32) {
      const int r = r0 + threadIdx.x;
      float lv = INFINITY;                                   // padding rows contribute 2^-inf = 0
      if (r < rows) {
        const int tok = p.n - p.w + r / p.G, h = g * p.G + r % p.G;
        lv = lse[static_cast<long long>(tok) * p.Hq + h] * 1.4426950408889634f;
      }
      sL[threadIdx.x] = lv;
    }
    __syncthreads();
    const int rmax = min(32, rows - r0);
    for (int r = part; r < rmax; r += 16) {
      const float4* qrow = reinterpret_cast<const float4*>(&sQ[r * D]);
      float s = 0.f;
#pragma unroll 8
      for (int c4 = 0; c4 < D / 4; ++c4) {
        const float4 a = qrow[c4], b = krow[c4];
        s = fmaf(a.x, b.x, s); s = fmaf(a.y, b.y, s); s = fmaf(a.z, b.z, s); s = fmaf(a.w, b.w, s);
      }
      acc += exp2f(s * p.scale_log2 - sL[r]);
    }
  }
  acc += __shfl_xor_sync(0xffffffffu, acc, 1);
  acc += __shfl_xor_sync(0xffffffffu, acc, 2);
  acc += __shfl_xor_sync(0xffffffffu, acc, 4);
  acc += __shfl_xor_sync(0xffffffffu, acc, 8);
  const int key = key0 + kj;
  if (part == 0 && key < p.n_cand) score[key] = acc;
  __syncthreads();
  if (threadIdx.x == 0) stamp_end(p);
}

// ------------------------------------------------------------------------------------------------
// Self-test of the bounded wait: one CTA waits on an mbarrier that nobody will ever arrive on.  With a wait limit
// of a few thousand cycles the wait gives up, the CTA passes its barrier, records KVC_ETIMEOUT in the status word
// exactly as the production kernels do, and returns.  Nothing in it can wait longer than the limit.
// grid 1, block 128.
__global__ void __launch_bounds__(128) wait_timeout_selftest_kernel(char* __restrict__ ws, int wait_limit_k) {
  __shared__ uint64_t bar;
  __shared__ int wait_ctl[2];
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    wait_ctl[0] = 0; wait_ctl[1] = wait_limit_k;
    mbar_fence_init();
  }
  __syncthreads();
  const bool ok = mbar_wait(&bar, 0, wait_ctl);          // phase 0 never completes: returns false after the limit
  __syncthreads();
  if (threadIdx.x == 0 && (!ok || wait_ctl[0])) atomicExch(reinterpret_cast<int*>(ws), -4 /* KVC_ETIMEOUT */);
}

}  // namespace kvc
