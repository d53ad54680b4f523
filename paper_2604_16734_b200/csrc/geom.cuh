// Launch geometry shared by every kernel of one kvc_prefill_chunk call.
#pragma once
#include <cuda_bf16.h>
#include <stdint.h>

namespace kvc {

// Notation follows the paper's Alg. 1: B is the memory budget M, n the block size b.
struct Geom {
  int n;          // tokens in this block
  int n_c;        // cache length before the block
  int tot;        // n_c + n (length right after "C <- C u (K_i, V_i)")
  int B;          // budget per (layer, kv-head)
  int w;          // observer window of this call = min(obs_window, n)
  int G, Hq, Hkv, d, cap, nl, max_chunk;
  int n_cand;     // tot - w : entries that compete for the budget
  int n_keep;     // B - w   : how many of them survive
  float scale_log2;           // softmax scale times log2(e): probabilities are 2^(s*scale_log2 - lse2)
  long long pos0;             // absolute position of the block's first token
  long long q_ls, kv_ls, out_ls;   // layer strides of q/out and k/v inputs, in elements
  long long cache_ls;              // layer stride of the cache blobs, bytes
  long long v_off, pos_off;        // byte offsets of V and pos inside a blob (K is at 0)
  long long ws_ls;                 // workspace slot stride, bytes (one slot per batched layer)
  int slot0;                       // workspace slot of the call's first layer (0 unless compress runs on the side stream)
  long long lse_off, score_off, msrc_off, mdst_off, mcount_off;   // byte offsets inside a slot
  int wait_limit_k;                // limit of every device-side wait, in units of 1024 clock cycles
  // measurement runs only (else null): this launch's pair of time stamps, {earliest begin of work, latest end} over
  // its CTAs, in nanoseconds of the global timer
  unsigned long long* stamps;
};

static constexpr int kNumSMs = 148;          // B200
static constexpr int kWsHeaderBytes = 256;   // status word lives at byte 0 of the workspace

// Device-side duration of a launch: a CTA stamps the begin of its work once it is past the wait for the preceding
// kernel, and its end when it is done; the launch's record keeps the minimum and the maximum.
__device__ __forceinline__ unsigned long long global_timer_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ void stamp_begin(const Geom& p) { if (p.stamps) atomicMin(p.stamps, global_timer_ns()); }
__device__ __forceinline__ void stamp_end(const Geom& p) { if (p.stamps) atomicMax(p.stamps + 1, global_timer_ns()); }

__device__ __forceinline__ char* ws_slot(char* ws, const Geom& p, int slot) {
  return ws + kWsHeaderBytes + static_cast<long long>(p.slot0 + slot) * p.ws_ls;
}

template <typename T> __device__ __forceinline__ float to_f32(T x);
template <> __device__ __forceinline__ float to_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 x) { return __bfloat162float(x); }
template <typename T> __device__ __forceinline__ T from_f32(float x);
template <> __device__ __forceinline__ float from_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float x) { return __float2bfloat16_rn(x); }

}  // namespace kvc
