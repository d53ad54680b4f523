// Host side of the kvc C ABI (see include/kvc.h): argument checks, launch geometry, TMA tensor
// maps, kernel launches on the caller's stream.  Allocates no device memory.
#include "../../include/kvc.h"

#include <cuda.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdarg.h>
#include <stdint.h>
#include <stdio.h>
#include <string.h>

#include <new>
#include <vector>

#include "geom.cuh"
#include "kernels_cc.cuh"
#include "kernels_tc.cuh"
#include "compress.cuh"

using kvc::Geom;

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct kvc_ctx {
  uint32_t magic;
  kvc_config cfg;
  int G, cap, w_cfg;
  float scale;
  size_t elem, blob_bytes, v_off, pos_off;
  size_t ws_slot_bytes, ws_bytes, lse_off, score_off, msrc_off, mdst_off, mcount_off;
  std::vector<int> len;          // current cache length per layer, -1 = never reset
  long long launches;
  EncodeTiledFn encode;
  bool use_tc;
  bool profiling;
  int wait_limit_k;              // limit of the kernels' waits, in units of 1024 clock cycles
  struct Prof { int kind; cudaEvent_t a, b; };
  std::vector<Prof> prof;
  // device-side time stamps (kvc_profile_device): the caller's record buffer, its capacity, the kind of every launch so far
  unsigned long long* stamps_dev;
  long long stamps_cap;
  std::vector<int> stamp_kind;
  // KVC_FLAG_ASYNC_COMPRESS: the side streams, per layer an event after its attention and one after its
  // compress kernel, and whether that compress may still be running (host objects, created on first use)
  static constexpr int kSideStreams = 2;     // layers alternate between them: consecutive compress kernels may overlap
  cudaStream_t side[kSideStreams];
  std::vector<cudaEvent_t> ev_attn, ev_comp;
  std::vector<char> pending;
  // kvc_prefill_chunk_host: the stream that carries the host-to-device copies, per staging half an event after its
  // copies (recorded there) and one after the block that read it (recorded on the caller's stream); call counter
  cudaStream_t copy_in, copy_out;
  cudaEvent_t ev_in[2], ev_free[2], ev_out[2];
  unsigned host_calls;
  char err[512];
};

static const uint32_t kMagic = 0x6b766331u;   // "kvc1"

static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

static int fail(kvc_ctx* c, int code, const char* fmt, ...) {
  if (c) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(c->err, sizeof(c->err), fmt, ap);
    va_end(ap);
  }
  return code;
}

static bool live(const kvc_ctx* c) { return c && c->magic == kMagic; }

extern "C" int kvc_create(const kvc_config* cfg, kvc_ctx** out) {
  if (!out) return KVC_EINVAL;
  *out = nullptr;
  if (!cfg) return KVC_EINVAL;
  if (cfg->n_layers < 1 || cfg->n_kv_heads < 1 || cfg->n_q_heads < 1) return KVC_EINVAL;
  if (cfg->n_q_heads % cfg->n_kv_heads != 0) return KVC_EINVAL;
  if (cfg->head_dim != 64 && cfg->head_dim != 128) return KVC_EINVAL;
  if (cfg->dtype != KVC_F32 && cfg->dtype != KVC_BF16) return KVC_EINVAL;
  if (cfg->budget < 1 || cfg->max_chunk < 1) return KVC_EINVAL;
  if (cfg->policy != KVC_SCORE_ATTN && cfg->policy != KVC_SCORE_KEYDIFF) return KVC_EINVAL;
  if (cfg->obs_window < 0) return KVC_EINVAL;
  if (!(cfg->softmax_scale >= 0.f) || isinf(cfg->softmax_scale)) return KVC_EINVAL;
  const int w = cfg->obs_window == 0 ? 32 : cfg->obs_window;
  if (w > cfg->budget) return KVC_EINVAL;                 // the protected window must fit the budget
  const int G = cfg->n_q_heads / cfg->n_kv_heads;
  if (G > 128) return KVC_EINVAL;
  if (cfg->device < 0 || cfg->device >= 64) return KVC_EINVAL;   // per-device tables below hold 64 ordinals
  if ((long long)cfg->budget + cfg->max_chunk > (1ll << 30)) return KVC_EINVAL;

  kvc_ctx* c = new (std::nothrow) kvc_ctx();
  if (!c) return KVC_EINVAL;
  c->magic = kMagic;
  c->cfg = *cfg;
  c->G = G;
  c->w_cfg = w;
  c->scale = cfg->softmax_scale > 0.f ? cfg->softmax_scale : 1.0f / sqrtf((float)cfg->head_dim);
  c->cap = (int)align_up((size_t)cfg->budget + cfg->max_chunk, 128);
  c->elem = cfg->dtype == KVC_F32 ? 4 : 2;
  const size_t kv_bytes = (size_t)cfg->n_kv_heads * c->cap * cfg->head_dim * c->elem;
  c->v_off = kv_bytes;
  c->pos_off = 2 * kv_bytes;
  c->blob_bytes = align_up(2 * kv_bytes + (size_t)cfg->n_kv_heads * c->cap * 4, 1024);
  size_t o = 0;
  // (lse has room for a first block of up to B tokens: the hybrid schedule of Sec. 5 (Budgeting) fills an empty cache in one pass)
  const size_t lse_rows = cfg->max_chunk > cfg->budget ? cfg->max_chunk : cfg->budget;
  c->lse_off = o;    o = align_up(o + lse_rows * cfg->n_q_heads * 4, 256);
  c->score_off = o;  o = align_up(o + (size_t)cfg->n_kv_heads * c->cap * 4, 256);
  c->msrc_off = o;   o = align_up(o + (size_t)cfg->n_kv_heads * cfg->max_chunk * 4, 256);
  c->mdst_off = o;   o = align_up(o + (size_t)cfg->n_kv_heads * cfg->max_chunk * 4, 256);
  c->mcount_off = o; o = align_up(o + (size_t)cfg->n_kv_heads * 4, 256);
  c->ws_slot_bytes = o;
  c->ws_bytes = kvc::kWsHeaderBytes + o * cfg->n_layers;
  c->len.assign(cfg->n_layers, -1);
  c->launches = 0;
  c->encode = nullptr;
  c->use_tc = cfg->dtype == KVC_BF16 && !(cfg->flags & KVC_FLAG_CUDA_CORES);
  c->profiling = false;
  c->stamps_dev = nullptr;
  c->stamps_cap = 0;
  c->wait_limit_k = kvc::kDefaultWaitLimitK;
  for (auto& s : c->side) s = nullptr;
  c->pending.assign(cfg->n_layers, 0);
  c->copy_in = c->copy_out = nullptr;
  for (int i = 0; i < 2; ++i) { c->ev_in[i] = nullptr; c->ev_free[i] = nullptr; c->ev_out[i] = nullptr; }
  c->host_calls = 0;
  c->err[0] = 0;
  *out = c;
  return KVC_OK;
}

static void drop_events(kvc_ctx* c) {
  for (auto& p : c->prof) { cudaEventDestroy(p.a); cudaEventDestroy(p.b); }
  c->prof.clear();
}

extern "C" int kvc_profile_enable(kvc_ctx* c, int on) {
  if (!live(c)) return KVC_ESTATE;
  c->profiling = on != 0;
  if (!on) drop_events(c);
  return KVC_OK;
}

extern "C" int kvc_profile_read(kvc_ctx* c, double* ms, long long* launches) {
  if (!live(c)) return KVC_ESTATE;
  if (!ms || !launches) return KVC_EINVAL;
  int rc = KVC_OK;
  for (auto& p : c->prof) {
    float t = 0.f;
    cudaError_t e = cudaEventSynchronize(p.b);
    if (e == cudaSuccess) e = cudaEventElapsedTime(&t, p.a, p.b);
    if (e != cudaSuccess) { rc = fail(c, KVC_ECUDA, "profile event: %s", cudaGetErrorString(e)); break; }
    ms[p.kind] += t;
    launches[p.kind] += 1;
  }
  drop_events(c);
  return rc;
}

extern "C" int kvc_profile_device(kvc_ctx* c, void* records, long long capacity, void* stream) {
  if (!live(c)) return KVC_ESTATE;
  c->stamp_kind.clear();
  c->stamps_dev = nullptr;
  c->stamps_cap = 0;
  if (!records) return KVC_OK;
  if (capacity < 1 || (reinterpret_cast<uintptr_t>(records) & 15)) return fail(c, KVC_EINVAL, "records misaligned or capacity < 1");
  // every record starts as {begin = all ones, end = 0}: the kernels keep the minimum and the maximum
  cudaError_t e = cudaMemsetAsync(records, 0, (size_t)capacity * 16, (cudaStream_t)stream);
  if (e == cudaSuccess) e = cudaMemset2DAsync(records, 16, 0xff, 8, (size_t)capacity, (cudaStream_t)stream);
  if (e != cudaSuccess) return fail(c, KVC_ECUDA, "cudaMemsetAsync(records): %s", cudaGetErrorString(e));
  c->stamps_dev = (unsigned long long*)records;
  c->stamps_cap = capacity;
  return KVC_OK;
}

extern "C" int kvc_profile_device_read(kvc_ctx* c, const void* records_host, double* ms, long long* launches, double* span_ms) {
  if (!live(c)) return KVC_ESTATE;
  if (!records_host || !ms || !launches) return KVC_EINVAL;
  const unsigned long long* r = (const unsigned long long*)records_host;
  unsigned long long first = ~0ull, last = 0;
  for (size_t i = 0; i < c->stamp_kind.size(); ++i) {
    const unsigned long long b = r[2 * i], e = r[2 * i + 1];
    if (b == ~0ull || e < b) continue;                    // a launch whose CTAs never stamped (nothing to do)
    ms[c->stamp_kind[i]] += (double)(e - b) * 1e-6;
    launches[c->stamp_kind[i]] += 1;
    if (b < first) first = b;
    if (e > last) last = e;
  }
  if (span_ms) *span_ms = last > first ? (double)(last - first) * 1e-6 : 0.0;
  c->stamp_kind.clear();
  return KVC_OK;
}

// The record of the next launch of the given kind (null when device stamps are off or the buffer is full).
static unsigned long long* next_stamp(kvc_ctx* c, int kind) {
  if (!c->stamps_dev || (long long)c->stamp_kind.size() >= c->stamps_cap) return nullptr;
  c->stamp_kind.push_back(kind);
  return c->stamps_dev + 2 * (c->stamp_kind.size() - 1);
}

// Brackets one kernel launch with events when profiling is on.
struct ProfScope {
  kvc_ctx* c; cudaStream_t st; cudaEvent_t a, b; bool on;
  ProfScope(kvc_ctx* c_, int kind, cudaStream_t st_) : c(c_), st(st_), a(nullptr), b(nullptr), on(c_->profiling) {
    if (!on) return;
    if (cudaEventCreate(&a) != cudaSuccess || cudaEventCreate(&b) != cudaSuccess) { on = false; return; }
    cudaEventRecord(a, st);
    c->prof.push_back({kind, a, b});
  }
  ~ProfScope() { if (on) cudaEventRecord(b, st); }
};

// Makes `st` wait for the compress kernels of layers [l0, l1) that still run on the side stream.
static int wait_pending(kvc_ctx* c, int l0, int l1, cudaStream_t st) {
  for (int l = l0; l < l1; ++l) {
    if (!c->pending[l]) continue;
    cudaError_t e = cudaStreamWaitEvent(st, c->ev_comp[l], 0);
    if (e != cudaSuccess) return fail(c, KVC_ECUDA, "cudaStreamWaitEvent: %s", cudaGetErrorString(e));
    c->pending[l] = 0;
  }
  return KVC_OK;
}

static int ensure_side_stream(kvc_ctx* c) {
  if (c->side[0]) return KVC_OK;                             // set last: marks a complete set of events and streams
  cudaError_t e = cudaSuccess;
  c->ev_attn.resize(c->cfg.n_layers, nullptr);
  c->ev_comp.resize(c->cfg.n_layers, nullptr);
  for (int l = 0; l < c->cfg.n_layers; ++l) {
    if (!c->ev_attn[l] && (e = cudaEventCreateWithFlags(&c->ev_attn[l], cudaEventDisableTiming)) != cudaSuccess) c->ev_attn[l] = nullptr;
    if (e == cudaSuccess && !c->ev_comp[l] && (e = cudaEventCreateWithFlags(&c->ev_comp[l], cudaEventDisableTiming)) != cudaSuccess) c->ev_comp[l] = nullptr;
    if (e != cudaSuccess) return fail(c, KVC_ECUDA, "cudaEventCreate: %s", cudaGetErrorString(e));
  }
  for (int i = kvc_ctx::kSideStreams - 1; i >= 0; --i) {
    if (c->side[i]) continue;
    if ((e = cudaStreamCreateWithFlags(&c->side[i], cudaStreamNonBlocking)) != cudaSuccess) {
      c->side[i] = nullptr;
      return fail(c, KVC_ECUDA, "cudaStreamCreate: %s", cudaGetErrorString(e));
    }
  }
  return KVC_OK;
}

extern "C" int kvc_join(kvc_ctx* c, void* stream) {
  if (!live(c)) return KVC_ESTATE;
  return wait_pending(c, 0, c->cfg.n_layers, (cudaStream_t)stream);
}

extern "C" int kvc_destroy(kvc_ctx* c) {
  if (!live(c)) return KVC_ESTATE;
  {
    for (auto s : c->side) if (s) cudaStreamSynchronize(s);
    for (auto ev : c->ev_attn) if (ev) cudaEventDestroy(ev);
    for (auto ev : c->ev_comp) if (ev) cudaEventDestroy(ev);
    c->ev_attn.clear(); c->ev_comp.clear();
    for (auto& s : c->side) { if (s) cudaStreamDestroy(s); s = nullptr; }
    if (c->copy_out) { cudaStreamSynchronize(c->copy_out); cudaStreamDestroy(c->copy_out); c->copy_out = nullptr; }
    if (c->copy_in) { cudaStreamSynchronize(c->copy_in); cudaStreamDestroy(c->copy_in); c->copy_in = nullptr; }
    for (int i = 0; i < 2; ++i) {
      if (c->ev_in[i]) cudaEventDestroy(c->ev_in[i]);
      if (c->ev_free[i]) cudaEventDestroy(c->ev_free[i]);
      if (c->ev_out[i]) cudaEventDestroy(c->ev_out[i]);
      c->ev_in[i] = c->ev_free[i] = c->ev_out[i] = nullptr;
    }
  }
  drop_events(c);
  c->magic = 0;
  delete c;
  return KVC_OK;
}

extern "C" const char* kvc_last_error(const kvc_ctx* c) { return live(c) ? c->err : "invalid context"; }
extern "C" long long kvc_launch_count(const kvc_ctx* c) { return live(c) ? c->launches : -1; }

extern "C" int kvc_cache_nbytes(const kvc_ctx* c, size_t* per_layer, size_t* workspace) {
  if (!live(c)) return KVC_ESTATE;
  if (per_layer) *per_layer = c->blob_bytes;
  if (workspace) *workspace = c->ws_bytes;
  return KVC_OK;
}

extern "C" int kvc_kv_bytes(const kvc_ctx* c, long long seq_len, size_t* logical, size_t* physical,
                            size_t* uncompressed) {
  if (!live(c)) return KVC_ESTATE;
  if (seq_len < 0) return KVC_EINVAL;
  // Eq. 2: 2 x layers x heads x dim_head x precision x sequence length
  const size_t per_tok = 2 * (size_t)c->cfg.n_layers * c->cfg.n_kv_heads * c->cfg.head_dim * c->elem;
  if (logical) *logical = per_tok * c->cfg.budget;
  if (physical) *physical = per_tok * c->cap;
  if (uncompressed) *uncompressed = per_tok * (size_t)seq_len;
  return KVC_OK;
}

static int check_cuda(kvc_ctx* c, cudaError_t e, const char* what) {
  if (e == cudaSuccess) return KVC_OK;
  return fail(c, KVC_ECUDA, "%s: %s", what, cudaGetErrorString(e));
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

extern "C" int kvc_reset(kvc_ctx* c, int layer, int n_layers, void* cache, size_t cache_layer_stride, void* stream) {
  if (!live(c)) return KVC_ESTATE;
  if (layer < 0 || n_layers < 1 || layer + n_layers > c->cfg.n_layers) return fail(c, KVC_EINVAL, "layer range");
  if (!cache || !aligned16(cache)) return fail(c, KVC_EINVAL, "cache pointer null or misaligned");
  if (n_layers > 1 && (cache_layer_stride < c->blob_bytes || cache_layer_stride % 16)) return fail(c, KVC_EINVAL, "cache_layer_stride");
  cudaStream_t st = (cudaStream_t)stream;
  if (int rc = wait_pending(c, layer, layer + n_layers, st)) return rc;
  for (int i = 0; i < n_layers; ++i) {
    int rc = check_cuda(c, cudaMemsetAsync((char*)cache + (size_t)i * cache_layer_stride, 0, c->blob_bytes, st), "cudaMemsetAsync");
    if (rc) return rc;
    c->len[layer + i] = 0;
  }
  return KVC_OK;
}

extern "C" int kvc_workspace_init(kvc_ctx* c, void* workspace, void* stream) {
  if (!live(c)) return KVC_ESTATE;
  if (!workspace || !aligned16(workspace)) return fail(c, KVC_EINVAL, "workspace pointer null or misaligned");
  return check_cuda(c, cudaMemsetAsync(workspace, 0, kvc::kWsHeaderBytes, (cudaStream_t)stream), "cudaMemsetAsync");
}

extern "C" int kvc_cache_view(const kvc_ctx* c, int layer, void* cache, kvc_view* v) {
  if (!live(c)) return KVC_ESTATE;
  if (!v || !cache || layer < 0 || layer >= c->cfg.n_layers) return KVC_EINVAL;
  if (c->len[layer] < 0) return KVC_ESTATE;
  v->k = cache;
  v->v = (char*)cache + c->v_off;
  v->pos = (int*)((char*)cache + c->pos_off);
  v->len = c->len[layer];
  v->cap = c->cap;
  v->n_kv_heads = c->cfg.n_kv_heads;
  v->head_dim = c->cfg.head_dim;
  v->dtype = c->cfg.dtype;
  return KVC_OK;
}

extern "C" int kvc_workspace_view(const kvc_ctx* c, void* workspace, int slot, float** lse, float** score) {
  if (!live(c)) return KVC_ESTATE;
  if (!workspace || slot < 0 || slot >= c->cfg.n_layers) return KVC_EINVAL;
  char* s = (char*)workspace + kvc::kWsHeaderBytes + (size_t)slot * c->ws_slot_bytes;
  if (lse) *lse = (float*)(s + c->lse_off);
  if (score) *score = (float*)(s + c->score_off);
  return KVC_OK;
}

extern "C" int kvc_move_counts(const kvc_ctx* c, void* workspace, int slot, int** counts) {
  if (!live(c)) return KVC_ESTATE;
  if (!workspace || !counts || slot < 0 || slot >= c->cfg.n_layers) return KVC_EINVAL;
  *counts = (int*)((char*)workspace + kvc::kWsHeaderBytes + (size_t)slot * c->ws_slot_bytes + c->mcount_off);
  return KVC_OK;
}

extern "C" int kvc_set_wait_limit(kvc_ctx* c, long long cycles) {
  if (!live(c)) return KVC_ESTATE;
  if (cycles < 1024 || cycles > (1ll << 40)) return fail(c, KVC_EINVAL, "wait limit %lld outside [1024, 2^40] cycles", cycles);
  c->wait_limit_k = (int)(cycles >> 10);
  return KVC_OK;
}

extern "C" int kvc_selftest_wait_timeout(kvc_ctx* c, void* workspace, void* stream) {
  if (!live(c)) return KVC_ESTATE;
  if (!workspace || !aligned16(workspace)) return fail(c, KVC_EINVAL, "workspace pointer null or misaligned");
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev != c->cfg.device)
    return fail(c, KVC_ESTATE, "current CUDA device %d is not the context's device %d", dev, c->cfg.device);
  // never more than about 2^21 cycles (a millisecond): the kernel exists to run into its limit
  const int limit_k = c->wait_limit_k < 2048 ? c->wait_limit_k : 2048;
  kvc::wait_timeout_selftest_kernel<<<1, 128, 0, (cudaStream_t)stream>>>((char*)workspace, limit_k);
  c->launches++;
  return check_cuda(c, cudaGetLastError(), "self-test launch");
}

extern "C" int kvc_status(kvc_ctx* c, void* workspace, void* stream) {
  if (!live(c)) return KVC_ESTATE;
  if (!workspace) return KVC_EINVAL;
  int word = 0;
  int rc = wait_pending(c, 0, c->cfg.n_layers, (cudaStream_t)stream);
  if (rc) return rc;
  rc = check_cuda(c, cudaMemcpyAsync(&word, workspace, sizeof(int), cudaMemcpyDeviceToHost, (cudaStream_t)stream), "cudaMemcpyAsync");
  if (rc) return rc;
  rc = check_cuda(c, cudaStreamSynchronize((cudaStream_t)stream), "cudaStreamSynchronize");
  if (rc) return rc;
  if (word != 0) return fail(c, word == KVC_ETIMEOUT ? KVC_ETIMEOUT : KVC_ECUDA, "device status word %d", word);
  return KVC_OK;
}

// ------------------------------------------------------------------------------------------------
static int get_encoder(kvc_ctx* c) {
  if (c->encode) return KVC_OK;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
  if (e != cudaSuccess || qres != cudaDriverEntryPointSuccess || !fn)
    return fail(c, KVC_ECUDA, "cuTensorMapEncodeTiled entry point unavailable: %s", cudaGetErrorString(e));
  c->encode = (EncodeTiledFn)fn;
  return KVC_OK;
}

// bf16 4-D tensor map with 128-byte swizzle; dims/box innermost first, strides in bytes for dims 1..3.
static int make_map(kvc_ctx* c, CUtensorMap* m, const void* base, const uint64_t dims[4], const uint64_t strides[3],
                    const uint32_t box[4]) {
  cuuint64_t gd[4] = {dims[0], dims[1], dims[2], dims[3]};
  cuuint64_t gs[3] = {strides[0], strides[1], strides[2]};
  cuuint32_t bx[4] = {box[0], box[1], box[2], box[3]};
  cuuint32_t es[4] = {1, 1, 1, 1};
  CUresult r = c->encode(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), gd, gs, bx, es,
                         CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS)
    return fail(c, KVC_ECUDA, "cuTensorMapEncodeTiled failed (%d): dims %llu %llu %llu %llu box %u %u %u %u", (int)r,
                (unsigned long long)dims[0], (unsigned long long)dims[1], (unsigned long long)dims[2],
                (unsigned long long)dims[3], box[0], box[1], box[2], box[3]);
  return KVC_OK;
}

// cudaFuncSetAttribute acts on the current device only: every kernel that opts into more dynamic shared memory keeps
// one flag per device ordinal (the caller has checked that the current device is the context's).
static const int kMaxDevices = 64;
template <typename Kernel>
static cudaError_t opt_in_smem(Kernel kernel, int bytes, bool* done_per_device, int dev) {
  if (done_per_device[dev]) return cudaSuccess;
  cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e == cudaSuccess) done_per_device[dev] = true;
  return e;
}

template <typename T, int D>
static void launch_cc_attn(const Geom& g, const void* q, void* cache, void* out, void* ws, cudaStream_t st) {
  dim3 grid((g.n + 15) / 16, g.Hq, g.nl);
  kvc::attn_cc_kernel<T, D><<<grid, 128, 0, st>>>((const T*)q, (const char*)cache, (T*)out, (char*)ws, g);
}
template <typename T, int D>
static cudaError_t launch_cc_score(const Geom& g, int dev, const void* q, void* cache, void* ws, cudaStream_t st) {
  const int smem = (kvc::kScoreCcKeys * (D + 4) + 32 * D + 32) * 4;
  static bool attr_set[kMaxDevices] = {};
  if (cudaError_t e = opt_in_smem(kvc::score_cc_kernel<T, D>, smem, attr_set, dev)) return e;
  dim3 grid((g.n_cand + kvc::kScoreCcKeys - 1) / kvc::kScoreCcKeys, g.Hkv, g.nl);
  kvc::score_cc_kernel<T, D><<<grid, 128, smem, st>>>((const T*)q, (const char*)cache, (char*)ws, g);
  return cudaSuccess;
}

// Launch attributes shared by the PDL-aware kernels: an optional cluster size and, unless disabled,
// programmatic stream serialization (the kernel may start while its predecessor drains; it calls
// griddepcontrol.wait before it touches anything the predecessor wrote or still reads).
struct LaunchAttrs {
  cudaLaunchAttribute at[2];
  int n;
  LaunchAttrs(int cluster_x, bool pdl) : n(0) {
    if (cluster_x > 0) {
      at[n].id = cudaLaunchAttributeClusterDimension;
      at[n].val.clusterDim.x = cluster_x; at[n].val.clusterDim.y = 1; at[n].val.clusterDim.z = 1;
      ++n;
    }
    if (pdl) {
      at[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
      at[n].val.programmaticStreamSerializationAllowed = 1;
      ++n;
    }
  }
};

// Number of CTAs the key range of one row-tile pair is split over (= cluster size): enough to put
// a CTA on every SM when the row tiles alone cannot, as long as every CTA keeps a few key tiles.
// (An exchange of the partials through an L2-resident global buffer instead of distributed shared
// memory was measured too: slower, the release / acquire round trip costs more than the narrow
// SM-to-SM path.)
// Launch shape of the tensor-core attention: R row tiles per CTA (1 or 2) and the key split S over a cluster.
// For each R the split is the largest that the SM count, the portable cluster size and the rule of three key
// tiles per CTA allow; the two candidates are then compared with a model of the kernel's duration fitted to
// in-kernel time stamps (us): a key tile costs 1.8 per pair of row tiles taking turns and 1.15 for a single
// tile (whose two softmax groups take alternate key tiles); the combine costs 3.5 for its barriers and the reduce plus 3.6 per row tile for the remote stores of a
// whole tile's partial rows; CTAs beyond one per SM run as further waves.
static void attn_launch_shape(const Geom& g, bool allow_split, int* S_out, int* R_out) {
  const int TOK = 128 / g.G;
  const int tiles = (g.n + TOK - 1) / TOK;
  const int T = (g.n_c + 127) / 128 + (g.n + 127) / 128;
  double best = 0.0;
  for (int R = 2; R >= 1; --R) {
    const long long base = (long long)((tiles + R - 1) / R) * g.Hkv * g.nl;
    int S = allow_split ? (int)(kvc::kNumSMs / base) : 1;
    if (S > 8) S = 8;                    // portable cluster size limit
    if (S > T / 3) S = T / 3;            // the exchange costs about as much as two key tiles: keep three per CTA
    while (S & (S - 1)) S &= S - 1;      // a power of two: the 128 rows of a tile divide evenly among the ranks
    if (S < 1) S = 1;
    const int Tl = (T + S - 1) / S;
    const long long waves = (base * S + kvc::kNumSMs - 1) / kvc::kNumSMs;
    double est = Tl * (R == 2 ? 1.8 : 1.15) * (double)waves;
    if (S > 1) est += 3.5 + R * 3.6 * (S - 1) / S;
    if (R == 2 || est < best) { best = est; *S_out = S; *R_out = R; }
    if (tiles == 1) break;               // a single row tile: both shapes are the same launch
  }
}

template <int D>
static cudaError_t launch_tc_attn(const Geom& g, int dev, const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv,
                                  const CUtensorMap& tkin, const CUtensorMap& tvin, void* cache, void* out, void* ws, int S,
                                  int R, bool pdl, cudaStream_t st) {
  const int smem = (2 + kvc::kStages) * (D / 64) * kvc::kSubTileBytes + 1024;
  static bool attr_set[kMaxDevices] = {};
  if (cudaError_t e = opt_in_smem(kvc::attn_tc_kernel<D>, smem, attr_set, dev)) return e;
  const int TOK = 128 / g.G;
  const int groups = ((g.n + TOK - 1) / TOK + R - 1) / R;
  cudaLaunchConfig_t lc;
  memset(&lc, 0, sizeof(lc));
  lc.gridDim = dim3(groups * S, g.Hkv, g.nl);
  lc.blockDim = dim3(kvc::kAttnThreads, 1, 1);
  lc.dynamicSmemBytes = smem;
  lc.stream = st;
  LaunchAttrs la(S, pdl);
  lc.attrs = la.at;
  lc.numAttrs = la.n;
  return cudaLaunchKernelEx(&lc, kvc::attn_tc_kernel<D>, tq, tk, tv, tkin, tvin, (char*)cache, (__nv_bfloat16*)out,
                            (char*)ws, g, S, R);
}
// a2..a4 fused (compress.cuh).  MODE: kvc::kScoresGiven / kScoreAttention / kScoreKeyDiff.
template <int D, int MODE>
static cudaError_t launch_compress(const Geom& g, int dev, const CUtensorMap& tk, const CUtensorMap& tqo, void* cache, void* ws,
                                   int elem_bytes, bool pdl, bool wide_ok, int cn_cap, cudaStream_t st) {
  const int score_bytes = MODE == kvc::kScoreAttention ? 2 * (D / 64) * kvc::kSubTileBytesC + (D / 64) * kvc::kMaxObsRowsFused * 128 : 0;
  const int table_bytes = kvc::kMaxKeysSmem * 8 + 2 * kvc::kMaxMovesSmem * 4 + 2 * kvc::kSelBins * 4;   // keys, move tables, histograms
  const int smem_min = (score_bytes > table_bytes ? score_bytes : table_bytes) + 1024;
  const int smem_solo = 120 * 1024;                      // more than half an SM: one CTA per SM
  static bool attr_set[kMaxDevices] = {};
  if (cudaError_t e = opt_in_smem(kvc::compress_kernel<D, MODE>, smem_solo, attr_set, dev)) return e;
  // Clusters of more than 8 CTAs are not portable: the kernel must allow them, and the device says how many clusters
  // of a size (one CTA per SM) it can hold at a time -- asked once per device and size; 0 where it refuses.
  static int wide_clusters[kMaxDevices][kvc::kMaxClusterWide + 1] = {};   // 0: not asked yet, -1: none, else clusters in flight
  auto clusters_in_flight = [&](int size) {
    int& slot = wide_clusters[dev][size];
    if (slot == 0) {
      int n_wide = 0;
      if (cudaFuncSetAttribute(kvc::compress_kernel<D, MODE>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) == cudaSuccess) {
        cudaLaunchConfig_t q;
        memset(&q, 0, sizeof(q));
        q.gridDim = dim3(size, 1, 1);
        q.blockDim = dim3(kvc::kCompressThreads, 1, 1);
        q.dynamicSmemBytes = smem_solo;
        LaunchAttrs qa(size, false);
        q.attrs = qa.at;
        q.numAttrs = qa.n;
        if (cudaOccupancyMaxActiveClusters(&n_wide, kvc::compress_kernel<D, MODE>, &q) != cudaSuccess) n_wide = 0;
      }
      (void)cudaGetLastError();                           // a refusal is an answer, not an error of this call
      slot = n_wide > 0 ? n_wide : -1;
    }
    return slot;
  };
  // cluster size: spread one kv-head over several SMs when the heads alone cannot fill the GPU
  const int n_tiles = (g.n_cand + 127) / 128;
  int Cn = (int)(kvc::kNumSMs / ((long long)g.Hkv * g.nl));
  if (Cn > kvc::kMaxClusterWide) Cn = kvc::kMaxClusterWide;
  // More than the portable 8 CTAs only while every cluster of the launch can be resident at once, and only in stream
  // order: on a side stream the kernel shares the GPU with the next layer's attention, where a wider cluster waits
  // longer for its SMs than it saves (measured: the video workload's step went from 44 to 49 ms).
  if (!wide_ok && Cn > 8) Cn = 8;
  if (cn_cap > 0 && Cn > cn_cap) Cn = cn_cap;             // (side stream: stay within the SMs the attention leaves idle)
  while (Cn > 8 && clusters_in_flight(Cn) < (long long)g.Hkv * g.nl) --Cn;
  const int tiles_per_cta = 2;                            // fewer, and the cluster barriers cost more than the tiles
  if (Cn > (n_tiles + tiles_per_cta - 1) / tiles_per_cta) Cn = (n_tiles + tiles_per_cta - 1) / tiles_per_cta;
  if (Cn < 1) Cn = 1;
  // Two CTAs share an SM only when there are more CTAs than SMs (then one scores while the other selects);
  // a launch that fits the GPU asks for more than half an SM's shared memory so that every CTA gets an SM
  // of its own instead of being packed in pairs.
  const int smem = (long long)Cn * g.Hkv * g.nl > kvc::kNumSMs ? smem_min : smem_solo;
  cudaLaunchConfig_t lc;
  memset(&lc, 0, sizeof(lc));
  lc.gridDim = dim3(Cn, g.Hkv, g.nl);
  lc.blockDim = dim3(kvc::kCompressThreads, 1, 1);
  lc.dynamicSmemBytes = smem;
  lc.stream = st;
  LaunchAttrs la(Cn, pdl);
  lc.attrs = la.at;
  lc.numAttrs = la.n;
  return cudaLaunchKernelEx(&lc, kvc::compress_kernel<D, MODE>, tk, tqo, (char*)cache, (char*)ws, g, Cn, elem_bytes);
}

template <int D>
static cudaError_t launch_tc_score(const Geom& g, int dev, const CUtensorMap& tk, const CUtensorMap& tqo, void* ws,
                                   int tok_per_group, cudaStream_t st) {
  const int smem = (D / 64) * (kvc::kSubTileBytes + 256 * 128) + 1024;
  static bool attr_set[kMaxDevices] = {};
  if (cudaError_t e = opt_in_smem(kvc::score_tc_kernel<D>, smem, attr_set, dev)) return e;
  dim3 grid((g.n_cand + 127) / 128, g.Hkv, g.nl);
  kvc::score_tc_kernel<D><<<grid, 128, smem, st>>>(tk, tqo, (char*)ws, g, tok_per_group);
  return cudaSuccess;
}

static int run_chunk(kvc_ctx* c, int layer0, int nl, const void* q, long long q_ls, const void* k, const void* v,
                     long long kv_ls, int n, long long pos0, void* cache, size_t cache_ls, void* ws, void* out,
                     long long out_ls, cudaStream_t st, int n_proxy = 0, bool allow_async = true,
                     bool clear_status = false) {
  const kvc_config& cf = c->cfg;
  if (layer0 < 0 || nl < 1 || layer0 + nl > cf.n_layers) return fail(c, KVC_EINVAL, "layer range [%d, %d) outside [0, %d)", layer0, layer0 + nl, cf.n_layers);
  if (!q || !k || !v || !cache || !ws || !out) return fail(c, KVC_EINVAL, "null pointer argument");
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(cache) || !aligned16(ws) || !aligned16(out))
    return fail(c, KVC_EINVAL, "pointers must be 16-byte aligned");
  // Blocks hold at most max_chunk tokens, except that an EMPTY cache may be filled with up to B tokens in one
  // pass (hybrid schedule, Sec. 5, Budgeting: the first M tokens go through in a single forward): nothing is evicted then.
  const int n_limit = (c->len[layer0] == 0 && cf.budget > cf.max_chunk) ? cf.budget : cf.max_chunk;
  if (n < 1 || n > n_limit) return fail(c, KVC_EINVAL, "n = %d outside [1, %d] (max_chunk = %d; up to B = %d into an empty cache)", n, n_limit, cf.max_chunk, cf.budget);
  if (pos0 < 0 || pos0 + n > 0x7fffffffLL) return fail(c, KVC_EINVAL, "pos0 out of range");
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev != cf.device)
    return fail(c, KVC_ESTATE, "current CUDA device %d is not the context's device %d", dev, cf.device);
  const int n_c = c->len[layer0];
  for (int i = 0; i < nl; ++i) {
    if (c->len[layer0 + i] < 0) return fail(c, KVC_ESTATE, "layer %d used before kvc_reset", layer0 + i);
    if (c->len[layer0 + i] != n_c) return fail(c, KVC_ESTATE, "batched layers hold different cache lengths");
  }
  if (nl > 1) {
    const long long qmin = (long long)n * cf.n_q_heads * cf.head_dim, kmin = (long long)n * cf.n_kv_heads * cf.head_dim;
    if (q_ls < qmin || out_ls < qmin || kv_ls < kmin || cache_ls < c->blob_bytes)
      return fail(c, KVC_EINVAL, "layer strides too small");
    if ((q_ls * c->elem) % 16 || (out_ls * c->elem) % 16 || (kv_ls * c->elem) % 16 || cache_ls % 16)
      return fail(c, KVC_EINVAL, "layer strides must be multiples of 16 bytes");
  } else {
    q_ls = out_ls = (long long)n * cf.n_q_heads * cf.head_dim;
    kv_ls = (long long)n * cf.n_kv_heads * cf.head_dim;
    cache_ls = c->blob_bytes;
  }

  Geom g;
  memset(&g, 0, sizeof(g));
  if (n_proxy < 0 || n_proxy >= n) return fail(c, KVC_EINVAL, "n_proxy = %d outside [0, n = %d)", n_proxy, n);
  // Proxy query tokens (the last n_proxy rows) are appended and attended like the rest of the block, but
  // the cache ends before them: rows tot .. tot + n_proxy are left behind as unused space, the proxies
  // are the observers, and with no protected window every entry competes for the B places.
  g.n = n; g.n_c = n_c; g.tot = n_c + n - n_proxy; g.B = cf.budget;
  g.w = n_proxy ? n_proxy : (c->w_cfg < n ? c->w_cfg : n);
  g.G = c->G; g.Hq = cf.n_q_heads; g.Hkv = cf.n_kv_heads; g.d = cf.head_dim; g.cap = c->cap; g.nl = nl;
  g.max_chunk = cf.max_chunk;
  g.n_cand = n_proxy ? g.tot : g.tot - g.w;
  g.n_keep = n_proxy ? g.B : g.B - g.w;
  g.scale_log2 = c->scale * 1.4426950408889634f;
  g.pos0 = pos0;
  g.q_ls = q_ls; g.kv_ls = kv_ls; g.out_ls = out_ls; g.cache_ls = (long long)cache_ls;
  g.v_off = (long long)c->v_off; g.pos_off = (long long)c->pos_off;
  g.ws_ls = (long long)c->ws_slot_bytes;
  // KVC_FLAG_ASYNC_COMPRESS: score / select / compact of a layer run on a side stream, beside whatever the caller
  // enqueues next (the next layer's attention, in a decoder stack, needs this layer's output, not its compacted
  // cache); the layer then works in its own workspace slot, and the next call that touches the layer waits
  const bool async_compress = (cf.flags & 16u) && nl == 1 && allow_async && c->use_tc;
  g.slot0 = async_compress ? layer0 : 0;
  g.lse_off = c->lse_off; g.score_off = c->score_off; g.msrc_off = c->msrc_off; g.mdst_off = c->mdst_off;
  g.mcount_off = c->mcount_off;
  g.wait_limit_k = c->wait_limit_k;
  const bool evict = g.tot > g.B;                      // Alg. 1: "if |C| > M"
  const bool f32 = cf.dtype == KVC_F32;
  const int D = cf.head_dim;

  // tensor maps first: nothing is enqueued if an encode fails
  CUtensorMap tq, tk, tv, tqo, tkin, tvin;
  int tok_per_group = 0;
  if (c->use_tc) {
    int rc = get_encoder(c);
    if (rc) return rc;
    const int TOK = 128 / g.G;
    const uint64_t qd[4] = {(uint64_t)D, (uint64_t)g.Hq, (uint64_t)n, (uint64_t)nl};
    const uint64_t qs[3] = {(uint64_t)D * 2, (uint64_t)g.Hq * D * 2, (uint64_t)q_ls * 2};
    const uint32_t qb[4] = {64, (uint32_t)g.G, (uint32_t)TOK, 1};
    if ((rc = make_map(c, &tq, q, qd, qs, qb))) return rc;
    const uint64_t kd[4] = {(uint64_t)D, (uint64_t)g.cap, (uint64_t)g.Hkv, (uint64_t)nl};
    const uint64_t ks[3] = {(uint64_t)D * 2, (uint64_t)g.cap * D * 2, (uint64_t)cache_ls};
    const uint32_t kb[4] = {64, 128, 1, 1};
    if ((rc = make_map(c, &tk, cache, kd, ks, kb))) return rc;
    if ((rc = make_map(c, &tv, (char*)cache + c->v_off, kd, ks, kb))) return rc;
    // the block's own keys / values, read in place: k, v are [n][Hkv][d]
    const uint64_t id[4] = {(uint64_t)D, (uint64_t)g.Hkv, (uint64_t)n, (uint64_t)nl};
    const uint64_t is[3] = {(uint64_t)D * 2, (uint64_t)g.Hkv * D * 2, (uint64_t)kv_ls * 2};
    const uint32_t ib[4] = {64, 1, 128, 1};
    if ((rc = make_map(c, &tkin, k, id, is, ib))) return rc;
    if ((rc = make_map(c, &tvin, v, id, is, ib))) return rc;
    if (evict) {
      tok_per_group = 256 / g.G;
      if (tok_per_group > g.w) tok_per_group = g.w;
      const uint32_t ob[4] = {64, (uint32_t)g.G, (uint32_t)tok_per_group, 1};
      if ((rc = make_map(c, &tqo, q, qd, qs, ob))) return rc;
    }
  }

  const bool pdl_main = !(cf.flags & 8u);              // flag 8: plain stream order between the kernels (diagnostic)
  const bool pdl = pdl_main;
  cudaError_t e = cudaSuccess;
  if (int rc = wait_pending(c, layer0, layer0 + nl, st)) return rc;    // a compress kernel of an earlier block may still run
  // every host check has passed: from here on work is enqueued.  A workspace that keeps an earlier user's contents
  // (the built-in scratch array) gets its status word cleared first.
  if (clear_status)
    if (int rc = check_cuda(c, cudaMemsetAsync(ws, 0, kvc::kWsHeaderBytes, st), "cudaMemsetAsync(status word)")) return rc;
  // a0 append (the tensor-core attention kernel appends by itself)
  if (!c->use_tc) {
    ProfScope ps(c, 0, st);
    g.stamps = next_stamp(c, 0);
    dim3 grid((n * g.Hkv + 7) / 8, 1, nl);
    cudaLaunchConfig_t lc;
    memset(&lc, 0, sizeof(lc));
    lc.gridDim = grid; lc.blockDim = dim3(256, 1, 1); lc.stream = st;
    LaunchAttrs la(0, pdl);
    lc.attrs = la.at; lc.numAttrs = la.n;
    if (f32) e = cudaLaunchKernelEx(&lc, kvc::append_kernel<float>, (const float*)k, (const float*)v, (char*)cache, g);
    else e = cudaLaunchKernelEx(&lc, kvc::append_kernel<__nv_bfloat16>, (const __nv_bfloat16*)k, (const __nv_bfloat16*)v, (char*)cache, g);
    c->launches++;
  }
  if (e != cudaSuccess) return check_cuda(c, e, "append launch");
  // a1 attention
  long long attn_ctas = 0;                                    // CTAs of the attention launch (tensor-core path)
  {
  ProfScope ps(c, 1, st);
  g.stamps = next_stamp(c, 1);
  if (c->use_tc) {
    int S = 1, R = 2;
    attn_launch_shape(g, !(cf.flags & 4u), &S, &R);
    const int TOK = 128 / g.G;
    attn_ctas = (long long)(((g.n + TOK - 1) / TOK + R - 1) / R) * S * g.Hkv * g.nl;
    e = D == 128 ? launch_tc_attn<128>(g, dev, tq, tk, tv, tkin, tvin, cache, out, ws, S, R, pdl, st)
                 : launch_tc_attn<64>(g, dev, tq, tk, tv, tkin, tvin, cache, out, ws, S, R, pdl, st);
  } else if (f32) {
    if (D == 128) launch_cc_attn<float, 128>(g, q, cache, out, ws, st); else launch_cc_attn<float, 64>(g, q, cache, out, ws, st);
  } else {
    if (D == 128) launch_cc_attn<__nv_bfloat16, 128>(g, q, cache, out, ws, st); else launch_cc_attn<__nv_bfloat16, 64>(g, q, cache, out, ws, st);
  }
  }
  if (e != cudaSuccess) return check_cuda(c, e, "attention launch setup");
  c->launches++;
  if (evict) {
    if (async_compress) {
      if (int rc = ensure_side_stream(c)) return rc;
      if ((e = cudaEventRecord(c->ev_attn[layer0], st)) != cudaSuccess || (e = cudaStreamWaitEvent(c->side[layer0 % kvc_ctx::kSideStreams], c->ev_attn[layer0], 0)) != cudaSuccess)
        return check_cuda(c, e, "side stream fork");
      st = c->side[layer0 % kvc_ctx::kSideStreams];                                           // everything below goes to the side stream
    }
    const bool pdl = pdl_main && !async_compress;             // an event, not a kernel, precedes the side stream's launches
    // On a side stream the kernel runs beside the next layer's attention, a launch of the same shape as this
    // layer's: a cluster per kv-head that fits the SMs that launch leaves idle shares nothing with it, while a wider
    // one takes SMs from attention CTAs, which then start late and lengthen the launch everything else waits for
    // (measured on the video workload: 44.3 -> 39.5 ms per step).
    int cn_cap = 0;
    if (async_compress && attn_ctas > 0 && kvc::kNumSMs - attn_ctas >= (long long)g.Hkv * g.nl) {
      const long long idle = kvc::kNumSMs - attn_ctas;
      cn_cap = (int)(idle / ((long long)g.Hkv * g.nl));
      // ... and a cluster must find its SMs inside one GPC, where the attention leaves about idle / 8 of them: a
      // cluster larger than that waits for attention CTAs to leave (tiled-image workload, 20 idle SMs, 4 kv-heads:
      // clusters of 4 or 5 CTAs 2.69e7 tokens/s/layer, of 3 or fewer 2.79e7).
      const int per_gpc = (int)((idle + 4) / 8);
      if (cn_cap > per_gpc) cn_cap = per_gpc > 0 ? per_gpc : 1;
    }
    const bool keydiff = cf.policy == KVC_SCORE_KEYDIFF;      // query-agnostic: always scored inside the fused kernel
    const bool fused_score = !keydiff && c->use_tc && g.w * g.G <= kvc::kMaxObsRowsFused;   // few observer rows: likewise
    if (!fused_score && !keydiff) {
      // a2 score as a kernel of its own (fp32 on CUDA cores; bf16 with more than 128 observer rows per kv-head:
      // fusing up to 256 rows was measured and is slower, the stand-alone kernel spreads the key tiles wider)
      ProfScope ps(c, 2, st);
      g.stamps = next_stamp(c, 2);
      if (c->use_tc) {
        e = D == 128 ? launch_tc_score<128>(g, dev, tk, tqo, ws, tok_per_group, st) : launch_tc_score<64>(g, dev, tk, tqo, ws, tok_per_group, st);
      } else if (f32) {
        e = D == 128 ? launch_cc_score<float, 128>(g, dev, q, cache, ws, st) : launch_cc_score<float, 64>(g, dev, q, cache, ws, st);
      } else {
        e = D == 128 ? launch_cc_score<__nv_bfloat16, 128>(g, dev, q, cache, ws, st) : launch_cc_score<__nv_bfloat16, 64>(g, dev, q, cache, ws, st);
      }
      if (e != cudaSuccess) return check_cuda(c, e, "score launch");
      c->launches++;
    }
    // (a2 +) a3 select + a4 compact
    {
      ProfScope ps(c, 3, st);
      g.stamps = next_stamp(c, 3);
      if (keydiff) e = launch_compress<64, kvc::kScoreKeyDiff>(g, dev, tk, tk, cache, ws, (int)c->elem, pdl, !async_compress, cn_cap, st);
      else if (fused_score) e = D == 128 ? launch_compress<128, kvc::kScoreAttention>(g, dev, tk, tqo, cache, ws, (int)c->elem, pdl, !async_compress, cn_cap, st)
                                         : launch_compress<64, kvc::kScoreAttention>(g, dev, tk, tqo, cache, ws, (int)c->elem, pdl, !async_compress, cn_cap, st);
      else e = launch_compress<64, kvc::kScoresGiven>(g, dev, tk, tk, cache, ws, (int)c->elem, pdl, !async_compress, cn_cap, st);
    }
    if (e != cudaSuccess) return check_cuda(c, e, "compress launch");
    c->launches++;
    if (async_compress) {
      if ((e = cudaEventRecord(c->ev_comp[layer0], st)) != cudaSuccess) return check_cuda(c, e, "side stream event");
      c->pending[layer0] = 1;
    }
  }
  int rc = check_cuda(c, cudaGetLastError(), "kernel launch");
  if (rc) return rc;
  const int new_len = evict ? g.B : g.tot;
  for (int i = 0; i < nl; ++i) c->len[layer0 + i] = new_len;
  return KVC_OK;
}

extern "C" int kvc_prefill_chunk(kvc_ctx* c, int layer, const void* q, const void* k, const void* v, int n,
                                 long long pos0, void* cache, void* workspace, void* out, void* stream) {
  if (!live(c)) return KVC_ESTATE;
  return run_chunk(c, layer, 1, q, 0, k, v, 0, n, pos0, cache, 0, workspace, out, 0, (cudaStream_t)stream);
}

extern "C" int kvc_prefill_chunk_proxy(kvc_ctx* c, int layer, const void* q, const void* k, const void* v, int n,
                                       int n_proxy, long long pos0, void* cache, void* workspace, void* out, void* stream) {
  if (!live(c)) return KVC_ESTATE;
  if (n_proxy < 1) return fail(c, KVC_EINVAL, "n_proxy = %d: at least one proxy token is needed (use kvc_prefill_chunk otherwise)", n_proxy);
  return run_chunk(c, layer, 1, q, 0, k, v, 0, n, pos0, cache, 0, workspace, out, 0, (cudaStream_t)stream, n_proxy);
}

extern "C" int kvc_prefill_chunk_layers(kvc_ctx* c, int layer0, int n_layers, const void* q, long long q_layer_stride,
                                        const void* k, const void* v, long long kv_layer_stride, int n, long long pos0,
                                        void* cache, size_t cache_layer_stride, void* workspace, void* out,
                                        long long out_layer_stride, void* stream) {
  if (!live(c)) return KVC_ESTATE;
  return run_chunk(c, layer0, n_layers, q, q_layer_stride, k, v, kv_layer_stride, n, pos0, cache, cache_layer_stride,
                   workspace, out, out_layer_stride, (cudaStream_t)stream);
}

// q, k, v and out of one block, each rounded up to 256 bytes
static size_t staging_half_bytes(size_t qb, size_t kb) { return 2 * align_up(qb, 256) + 2 * align_up(kb, 256); }

extern "C" int kvc_staging_nbytes(const kvc_ctx* c, size_t* nbytes) {
  if (!live(c)) return KVC_ESTATE;
  if (!nbytes) return KVC_EINVAL;
  const size_t rows = c->cfg.max_chunk > c->cfg.budget ? c->cfg.max_chunk : c->cfg.budget;   // room for a bulk first block
  const size_t qb = rows * c->cfg.n_q_heads * c->cfg.head_dim * c->elem;
  const size_t kb = rows * c->cfg.n_kv_heads * c->cfg.head_dim * c->elem;
  *nbytes = 2 * staging_half_bytes(qb, kb);                  // two halves: the copies of one block run beside the previous block
  return KVC_OK;
}

static int ensure_copy_stream(kvc_ctx* c) {
  if (c->copy_in) return KVC_OK;                             // set last: marks a complete set
  cudaError_t e = cudaSuccess;
  for (int i = 0; i < 2 && e == cudaSuccess; ++i) {
    if (!c->ev_in[i] && (e = cudaEventCreateWithFlags(&c->ev_in[i], cudaEventDisableTiming)) != cudaSuccess) c->ev_in[i] = nullptr;
    if (e == cudaSuccess && !c->ev_free[i] && (e = cudaEventCreateWithFlags(&c->ev_free[i], cudaEventDisableTiming)) != cudaSuccess) c->ev_free[i] = nullptr;
    if (e == cudaSuccess && !c->ev_out[i] && (e = cudaEventCreateWithFlags(&c->ev_out[i], cudaEventDisableTiming)) != cudaSuccess) c->ev_out[i] = nullptr;
  }
  if (e != cudaSuccess) return fail(c, KVC_ECUDA, "cudaEventCreate: %s", cudaGetErrorString(e));
  if (!c->copy_out && (e = cudaStreamCreateWithFlags(&c->copy_out, cudaStreamNonBlocking)) != cudaSuccess) {
    c->copy_out = nullptr;
    return fail(c, KVC_ECUDA, "cudaStreamCreate: %s", cudaGetErrorString(e));
  }
  if ((e = cudaStreamCreateWithFlags(&c->copy_in, cudaStreamNonBlocking)) != cudaSuccess) {
    c->copy_in = nullptr;
    return fail(c, KVC_ECUDA, "cudaStreamCreate: %s", cudaGetErrorString(e));
  }
  return KVC_OK;
}

extern "C" int kvc_prefill_chunk_host(kvc_ctx* c, int layer, const void* q_host, const void* k_host, const void* v_host,
                                      int n, long long pos0, void* cache, void* workspace, void* staging, void* out_host,
                                      void* stream) {
  if (!live(c)) return KVC_ESTATE;
  if (!q_host || !k_host || !v_host || !out_host || !staging) return fail(c, KVC_EINVAL, "null pointer argument");
  if (layer < 0 || layer >= c->cfg.n_layers) return fail(c, KVC_EINVAL, "layer %d outside [0, %d)", layer, c->cfg.n_layers);
  const int n_limit = (c->len[layer] == 0 && c->cfg.budget > c->cfg.max_chunk) ? c->cfg.budget : c->cfg.max_chunk;
  if (n < 1 || n > n_limit) return fail(c, KVC_EINVAL, "n = %d outside [1, %d]", n, n_limit);
  if (!aligned16(staging)) return fail(c, KVC_EINVAL, "staging must be 16-byte aligned");
  cudaStream_t st = (cudaStream_t)stream;
  const size_t qb = (size_t)n * c->cfg.n_q_heads * c->cfg.head_dim * c->elem;
  const size_t kb = (size_t)n * c->cfg.n_kv_heads * c->cfg.head_dim * c->elem;
  size_t total = 0;
  kvc_staging_nbytes(c, &total);
  int rc = ensure_copy_stream(c);
  if (rc) return rc;
  // Calls alternate between the two halves of the staging buffer.  The inputs travel on the context's inbound copy
  // stream, behind the block that last read this half (two calls ago); the caller's stream waits for them and runs
  // the block; `out` goes back on the context's outbound copy stream, behind the block.  So the inbound copies of
  // call i+1, the kernels of call i+1 (other half) and the outbound copy of call i all run at the same time.  The
  // caller's stream then waits for the outbound copy of the PREVIOUS call (the other half: its `out` area is the
  // next block's), which has had this call's kernels to finish.
  const int half = (int)(c->host_calls++ & 1u);
  char* dq = (char*)staging + half * (total / 2);
  char* dk = dq + align_up(qb, 256);
  char* dv = dk + align_up(kb, 256);
  char* dout = dv + align_up(kb, 256);
  if ((rc = check_cuda(c, cudaStreamWaitEvent(c->copy_in, c->ev_free[half], 0), "cudaStreamWaitEvent"))) return rc;
  if ((rc = check_cuda(c, cudaMemcpyAsync(dq, q_host, qb, cudaMemcpyHostToDevice, c->copy_in), "H2D q"))) return rc;
  if ((rc = check_cuda(c, cudaMemcpyAsync(dk, k_host, kb, cudaMemcpyHostToDevice, c->copy_in), "H2D k"))) return rc;
  if ((rc = check_cuda(c, cudaMemcpyAsync(dv, v_host, kb, cudaMemcpyHostToDevice, c->copy_in), "H2D v"))) return rc;
  if ((rc = check_cuda(c, cudaEventRecord(c->ev_in[half], c->copy_in), "cudaEventRecord"))) return rc;
  if ((rc = check_cuda(c, cudaStreamWaitEvent(st, c->ev_in[half], 0), "cudaStreamWaitEvent"))) return rc;
  rc = run_chunk(c, layer, 1, dq, 0, dk, dv, 0, n, pos0, cache, 0, workspace, dout, 0, st, 0, false);   // staging is reused: no side stream
  if (rc) return rc;
  if ((rc = check_cuda(c, cudaEventRecord(c->ev_free[half], st), "cudaEventRecord"))) return rc;
  if ((rc = check_cuda(c, cudaStreamWaitEvent(c->copy_out, c->ev_free[half], 0), "cudaStreamWaitEvent"))) return rc;
  if ((rc = check_cuda(c, cudaMemcpyAsync(out_host, dout, qb, cudaMemcpyDeviceToHost, c->copy_out), "D2H out"))) return rc;
  if ((rc = check_cuda(c, cudaEventRecord(c->ev_out[half], c->copy_out), "cudaEventRecord"))) return rc;
  // (an event that was never recorded counts as complete: the first call waits for nothing here)
  return check_cuda(c, cudaStreamWaitEvent(st, c->ev_out[1 - half], 0), "cudaStreamWaitEvent");
}

extern "C" int kvc_host_flush(kvc_ctx* c, void* stream) {
  if (!live(c)) return KVC_ESTATE;
  if (!c->copy_out) return KVC_OK;                           // no host call yet
  for (int i = 0; i < 2; ++i)
    if (int rc = check_cuda(c, cudaStreamWaitEvent((cudaStream_t)stream, c->ev_out[i], 0), "cudaStreamWaitEvent")) return rc;
  return KVC_OK;
}

// ------------------------------------------------------------------------------------------------
// Allocation-free variant: the scratch area is a fixed device array compiled into the library.
// In host code `g_static_ws` is only a handle for the runtime, not a device address; the address
// each device gives it is looked up once per device and cached here.
static __device__ __align__(256) unsigned char g_static_ws[KVC_STATIC_WS_BYTES];
static void* g_static_ws_ptr[kMaxDevices] = {nullptr};

static int static_ws_for_current_device(kvc_ctx* c, void** ptr) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return check_cuda(c, e, "cudaGetDevice");
  if (dev < 0 || dev >= kMaxDevices) return fail(c, KVC_EINVAL, "device ordinal %d not supported by the static scratch", dev);
  if (dev != c->cfg.device) return fail(c, KVC_ESTATE, "current CUDA device %d is not the context's device %d", dev, c->cfg.device);
  if (!g_static_ws_ptr[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_static_ws);
    if (e != cudaSuccess || !p) return check_cuda(c, e == cudaSuccess ? cudaErrorInvalidSymbol : e, "cudaGetSymbolAddress(static scratch)");
    g_static_ws_ptr[dev] = p;
  }
  *ptr = g_static_ws_ptr[dev];
  return KVC_OK;
}

extern "C" int kvc_prefill_chunk_static(kvc_ctx* c, int layer, const void* q, const void* k, const void* v, int n,
                                        long long pos0, void* cache, void* out, void* stream) {
  if (!live(c)) return KVC_ESTATE;
  if (c->profiling) return fail(c, KVC_ESTATE, "kvc_prefill_chunk_static needs profiling off");
  const size_t need = kvc::kWsHeaderBytes + c->ws_slot_bytes;          // header + one layer slot
  if (need > (size_t)KVC_STATIC_WS_BYTES)
    return fail(c, KVC_EINVAL, "configuration needs %zu bytes of scratch, the built-in scratch holds %u", need,
                (unsigned)KVC_STATIC_WS_BYTES);
  void* ws = nullptr;
  int rc = static_ws_for_current_device(c, &ws);
  if (rc) return rc;
  // the array keeps the previous call's contents: only the status word has to start at zero, and it is cleared
  // once the argument and state checks have passed (a rejected call enqueues nothing)
  return run_chunk(c, layer, 1, q, 0, k, v, 0, n, pos0, cache, 0, ws, out, 0, (cudaStream_t)stream, 0, false, true);
}

extern "C" int kvc_status_static(kvc_ctx* c, void* stream) {
  if (!live(c)) return KVC_ESTATE;
  void* ws = nullptr;
  int rc = static_ws_for_current_device(c, &ws);
  if (rc) return rc;
  return kvc_status(c, ws, stream);
}
