// lacache_full_recompute_static: plain attention for ONE sequence with no
// device allocation anywhere on the call path.
//
// Who needs this: code that runs where cudaMalloc is off limits -- inside a
// memory pool or arena that owns the whole device heap, in a plugin whose host
// forbids allocation after start-up, or in a latency-critical section where an
// allocation (an implicit device synchronisation) is not acceptable.  Such a
// caller cannot create a context (creating one allocates the caches), so this
// entry point keeps every piece of scratch the computation needs -- rotated
// q/k/v planes, the RoPE tables, token positions and the work list -- in one
// fixed array that lives in the library's device image.
#include <math.h>
#include <stdio.h>
#include <string.h>

#include "lacache_internal.h"

namespace lacache {
void set_thread_error(const char* msg);  // lacache_api.cu: text behind lacache_last_error(NULL)
}

using namespace lacache;

namespace {

// Fixed scratch: 4 Mi floats of rotated planes plus tables and metadata (18 MiB
// in all, held by every GPU that loads the library until the process exits).
constexpr size_t STATIC_MAX_PLANE_ELEMS = (size_t)4 << 20;  // T * (Hq + 2 Hkv) * d
constexpr int STATIC_MAX_TOKENS = 4096;
constexpr size_t STATIC_TABLE_ELEMS = (size_t)STATIC_MAX_TOKENS * 64 * 2;      // cos + sin, d/2 <= 64
constexpr size_t STATIC_META_WORDS = STATIC_MAX_TOKENS + 16 + (STATIC_MAX_TOKENS / SIMT_ROWS + 1) * 12;
constexpr size_t STATIC_WORDS = STATIC_MAX_PLANE_ELEMS + STATIC_TABLE_ELEMS + STATIC_META_WORDS;

static __device__ __align__(256) float g_static_scratch[STATIC_WORDS];

constexpr int MAX_DEVICES = 64;
float* g_scratch_dev[MAX_DEVICES];  // device address of the array, per device (nullptr = not set up)
// What the tables and metadata in a device's copy of the array were last filled for: a call with the same
// (n_tokens, head_dim, rope_theta) finds them as it needs them and copies nothing.
struct Filled { int n_tokens, head_dim; float theta; };
Filled g_filled[MAX_DEVICES];

// host-side staging for the tables and metadata (no allocation per call)
float h_cos[STATIC_MAX_TOKENS * 64];
float h_sin[STATIC_MAX_TOKENS * 64];
int32_t h_meta[STATIC_META_WORDS];

lacache_status fail(lacache_status st, const char* fmt, long long a = 0, long long b = 0) {
  char buf[256];
  snprintf(buf, sizeof(buf), fmt, a, b);
  set_thread_error(buf);
  return st;
}

}  // namespace

extern "C" lacache_status lacache_full_recompute_static(int dtype, int n_tokens, int n_q_heads, int n_kv_heads,
                                                        int head_dim, float rope_theta, float softmax_scale,
                                                        const void* q_pre, const void* k_pre, const void* v_pre,
                                                        float* out, float* lse, void* cuda_stream) {
  if (dtype != LACACHE_DTYPE_BF16 && dtype != LACACHE_DTYPE_FP32) return fail(LACACHE_ERR_UNSUPPORTED, "dtype %lld", dtype);
  if (head_dim != 64 && head_dim != 128) return fail(LACACHE_ERR_UNSUPPORTED, "head_dim %lld (64 or 128)", head_dim);
  if (n_q_heads < 1 || n_kv_heads < 1 || n_q_heads % n_kv_heads)
    return fail(LACACHE_ERR_SHAPE, "n_q_heads %lld not a multiple of n_kv_heads %lld", n_q_heads, n_kv_heads);
  if (n_tokens < 1) return fail(LACACHE_ERR_SHAPE, "n_tokens %lld < 1", n_tokens);
  if (!(rope_theta > 0.f)) return fail(LACACHE_ERR_INVALID_ARG, "rope_theta must be > 0");
  if (!q_pre || !k_pre || !v_pre || !out) return fail(LACACHE_ERR_INVALID_ARG, "NULL pointer");
  const uintptr_t bits = (uintptr_t)q_pre | (uintptr_t)k_pre | (uintptr_t)v_pre | (uintptr_t)out | (uintptr_t)lse;
  if (bits & 15u) return fail(LACACHE_ERR_INVALID_ARG, "pointer not 16-byte aligned");
  const size_t plane_elems = (size_t)n_tokens * (n_q_heads + 2 * n_kv_heads) * head_dim;
  if (n_tokens > STATIC_MAX_TOKENS)
    return fail(LACACHE_ERR_SHAPE, "n_tokens %lld exceeds the static scratch limit of %lld tokens", n_tokens, STATIC_MAX_TOKENS);
  if (plane_elems > STATIC_MAX_PLANE_ELEMS)
    return fail(LACACHE_ERR_SHAPE, "n_tokens * (n_q_heads + 2 n_kv_heads) * head_dim = %lld exceeds the static scratch limit of %lld elements",
                (long long)plane_elems, (long long)STATIC_MAX_PLANE_ELEMS);

  // ---- once per device: resolve the array's device address ----
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return fail(LACACHE_ERR_CUDA, cudaGetErrorString(e));
  if (dev < 0 || dev >= MAX_DEVICES) return fail(LACACHE_ERR_UNSUPPORTED, "device index %lld", dev);
  if (!g_scratch_dev[dev]) {
    // In host code the array's name is only a handle; the device address comes
    // from the runtime, for the device that is current right now.
    float* p = nullptr;
    e = cudaGetSymbolAddress((void**)&p, g_static_scratch);
    if (e != cudaSuccess || !p) return fail(LACACHE_ERR_CUDA, cudaGetErrorString(e));
    e = simt_prepare();
    if (e != cudaSuccess) return fail(LACACHE_ERR_CUDA, cudaGetErrorString(e));
    g_scratch_dev[dev] = p;
  }
  float* base = g_scratch_dev[dev];
  cudaStream_t s = (cudaStream_t)cuda_stream;

  // ---- carve the array ----
  Geometry g{};
  g.B = 1; g.T = n_tokens; g.Tp = n_tokens; g.maxN = n_tokens;
  g.Hq = n_q_heads; g.Hkv = n_kv_heads; g.d = head_dim; g.group = n_q_heads / n_kv_heads;
  g.gen_len = n_tokens; g.block_len = n_tokens; g.n_blk = 1;
  const double scale = softmax_scale > 0.f ? (double)softmax_scale : 1.0 / sqrt((double)head_dim);
  g.scale_log2 = (float)(scale * 1.4426950408889634074);
  const size_t nq = (size_t)n_q_heads * n_tokens * head_dim, nk = (size_t)n_kv_heads * n_tokens * head_dim;
  const int half = head_dim / 2;
  float* q_rot = base;
  float* k_rot = q_rot + nq;
  float* v_cpy = k_rot + nk;
  float* d_cos = base + STATIC_MAX_PLANE_ELEMS;
  float* d_sin = d_cos + (size_t)STATIC_MAX_TOKENS * 64;
  int32_t* d_meta = reinterpret_cast<int32_t*>(base + STATIC_MAX_PLANE_ELEMS + STATIC_TABLE_ELEMS);
  // meta: [0, T) positions | [T, T+16) cu (padded) | work items
  const int n_items = (n_tokens + SIMT_ROWS - 1) / SIMT_ROWS;
  const size_t items_off = ((size_t)n_tokens + 16 + 3) & ~(size_t)3;  // 16-byte aligned
  Filled& filled = g_filled[dev];
  const bool refill = filled.n_tokens != n_tokens || filled.head_dim != head_dim || filled.theta != rope_theta;
  if (refill) {
    filled.n_tokens = 0;   // (until the copies below are enqueued)
    for (int t = 0; t < n_tokens; ++t) h_meta[t] = t;
    memset(h_meta + n_tokens, 0, sizeof(int32_t) * 16);
    h_meta[n_tokens + 1] = n_tokens;  // cu = {0, T}
    WorkItem* items = reinterpret_cast<WorkItem*>(h_meta + items_off);
    for (int i = 0; i < n_items; ++i) {
      WorkItem w{};
      w.kind = ITEM_ROWS; w.seq = 0; w.row0 = i * SIMT_ROWS;
      w.nrows = n_tokens - w.row0 < SIMT_ROWS ? n_tokens - w.row0 : SIMT_ROWS;
      w.pad = 1; w.seq_start = 0; w.seq_end = n_tokens;
      items[i] = w;
    }
    for (int c = 0; c < half; ++c) {
      const double f = pow((double)rope_theta, -2.0 * (double)c / (double)head_dim);
      for (int p = 0; p < n_tokens; ++p) {
        const double ang = (double)p * f;
        h_cos[(size_t)p * half + c] = (float)cos(ang);
        h_sin[(size_t)p * half + c] = (float)sin(ang);
      }
    }
    // Nothing in the array has to start at zero: every word a kernel reads below
    // is written first by these copies or by the rotation kernel.
    const size_t meta_words = items_off + (size_t)n_items * (sizeof(WorkItem) / 4);
    if ((e = cudaMemcpyAsync(d_cos, h_cos, sizeof(float) * n_tokens * half, cudaMemcpyHostToDevice, s)) != cudaSuccess ||
        (e = cudaMemcpyAsync(d_sin, h_sin, sizeof(float) * n_tokens * half, cudaMemcpyHostToDevice, s)) != cudaSuccess ||
        (e = cudaMemcpyAsync(d_meta, h_meta, sizeof(int32_t) * meta_words, cudaMemcpyHostToDevice, s)) != cudaSuccess)
      return fail(LACACHE_ERR_CUDA, cudaGetErrorString(e));
    filled = Filled{n_tokens, head_dim, rope_theta};
  }

  RopeArgs r{};
  r.q = q_pre; r.k = k_pre; r.v = v_pre;
  r.n_src_rows = n_tokens;
  r.blk_start = nullptr; r.block_len = n_tokens;
  r.pos_of_tok = d_meta; r.cos_tab = d_cos; r.sin_tab = d_sin;
  r.dst = RotBuffers{q_rot, nullptr, k_rot, nullptr, v_cpy};
  r.in_dtype = dtype;
  if ((e = rope_write(g, r, LACACHE_ENGINE_SIMT, s)) != cudaSuccess) return fail(LACACHE_ERR_CUDA, cudaGetErrorString(e));

  AttnArgs a{};
  a.mode = MODE_FULL;
  a.items = reinterpret_cast<const WorkItem*>(d_meta + items_off);
  a.n_items = n_items;
  a.cu = d_meta + n_tokens;
  a.blk_start = nullptr;
  a.rot = r.dst;
  a.out = out;
  a.lse = lse;
  if ((e = simt_attention(g, a, s)) != cudaSuccess) return fail(LACACHE_ERR_CUDA, cudaGetErrorString(e));
  return LACACHE_OK;
}
