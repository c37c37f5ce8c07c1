// Sampling-stage truncation (Sec. 3.4, last paragraph): the float softmax over the vocabulary runs on
// the rows of the current block only.  Per block row: the most probable token (lowest id among equal
// logits), its probability and the log normaliser.  HBM-bound: every logit of the block's rows is read
// once, nothing else of the [T, vocab] array is touched.
//
// A row is cut into `splits` slices of the vocabulary, one CTA each (a block has few rows: one CTA per
// row would leave most SMs idle).  A CTA reduces its slice to (max, sum of exp relative to that max,
// index of the first maximum) with one pass and one exponential per element; the last CTA of a row to
// arrive (one counter per row, reset by that CTA) combines the slices in slice order, so the result
// does not depend on the arrival order.
#include <cuda_bf16.h>

#include "lacache_internal.h"

namespace lacache {
namespace {

constexpr int SAMPLE_THREADS = 256;
constexpr float LOG2E = 1.4426950408889634f;
constexpr float LN2F = 0.69314718055994531f;

struct Acc {
  float m, s;   // running maximum; sum of 2^((x - m) log2 e) over the elements seen
  int idx;      // index of the first element equal to m
};

__device__ __forceinline__ float ex2f(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ void acc_add(Acc& a, float x, int i) {
  if (x > a.m) {   // (strict: an equal logit further on does not move the index)
    a.s = a.s * ex2f((a.m - x) * LOG2E) + 1.f;
    a.m = x;
    a.idx = i;
  } else if (x != -INFINITY) {   // (a masked vocabulary entry adds nothing, also before any finite logit)
    a.s += ex2f((x - a.m) * LOG2E);
  }
}
// a and b cover disjoint index ranges
__device__ __forceinline__ Acc acc_merge(const Acc& a, const Acc& b) {
  Acc r;
  if (b.m > a.m || (b.m == a.m && b.idx < a.idx)) {
    r.m = b.m; r.idx = b.idx;
  } else {
    r.m = a.m; r.idx = a.idx;
  }
  const float sa = a.m == -INFINITY ? 0.f : a.s * ex2f((a.m - r.m) * LOG2E);
  const float sb = b.m == -INFINITY ? 0.f : b.s * ex2f((b.m - r.m) * LOG2E);
  r.s = sa + sb;
  return r;
}

// NV vectors of VEC elements each (vector u starts at index i0 + u * step) added without a per-element
// branch or rescale: maximum and its first index (compare + selects), one rescale of the sum, then one
// exponential per element.
template <int NV, int VEC>
__device__ __forceinline__ void batch_add(Acc& acc, const float (&f)[NV * VEC], int i0, int step) {
  float best = acc.m;
  int bidx = acc.idx;
#pragma unroll
  for (int u = 0; u < NV; ++u) {
#pragma unroll
    for (int j = 0; j < VEC; ++j) {
      const bool up = f[u * VEC + j] > best;   // (strict: an equal logit further on does not move the index)
      best = up ? f[u * VEC + j] : best;
      bidx = up ? i0 + u * step + j : bidx;
    }
  }
  const float m_use = best == -INFINITY ? 0.f : best;   // (only -inf so far: every term below is 0)
  float sum = acc.m == -INFINITY ? 0.f : acc.s * ex2f((acc.m - m_use) * LOG2E);
#pragma unroll
  for (int k = 0; k < NV * VEC; ++k) sum += ex2f((f[k] - m_use) * LOG2E);
  acc.m = best; acc.idx = bidx; acc.s = sum;
}

__device__ __forceinline__ float to_float(float x) { return x; }
__device__ __forceinline__ float to_float(__nv_bfloat16 x) { return __bfloat162float(x); }

template <class T>
__global__ void __launch_bounds__(SAMPLE_THREADS, 4) sample_rows_kernel(SampleArgs a) {
  constexpr int VEC = 16 / (int)sizeof(T);
  const int r = blockIdx.y, sp = blockIdx.x;
  const int row = a.rows[r];
  __shared__ Acc warp_acc[SAMPLE_THREADS / 32];
  const bool bad = row < 0 || row >= a.n_tokens;
  Acc acc{-INFINITY, 0.f, 0x7fffffff};
  if (!bad) {
    const T* x = reinterpret_cast<const T*>(a.logits) + (size_t)row * a.vocab;
    const int lo = sp * a.slice, hi = min(lo + a.slice, a.vocab);
    if (a.vector_ok) {   // rows start on 16-byte boundaries and the slice is a multiple of the vector width
      const int hi_v = lo + (max(hi - lo, 0) / VEC) * VEC;
      // Four independent 16-byte loads in flight per thread, then two batches of two vectors each
      // (batch_add: the lanes of a warp move their running maxima at different elements, so a
      // per-element branch would run both of its sides -- two exponentials, and the exponential
      // unit is what bounds this kernel -- nearly every time).  A slice is often shorter than four
      // vectors per thread (a block of 32 rows on 148 SMs gets ~18 slices of ~7000 entries a row): the
      // vectors past its end are filled with -inf, which adds nothing, so that the loads a thread does
      // have still leave together instead of one round trip after the other.
      constexpr int STEP = SAMPLE_THREADS * VEC;
      const uint32_t ninf = sizeof(T) == 2 ? 0xFF80FF80u : 0xFF800000u;
      for (int i = lo + threadIdx.x * VEC; i < hi_v; i += 4 * STEP) {
        uint4 raw[4];
#pragma unroll
        for (int u = 0; u < 4; ++u)
          raw[u] = (i + u * STEP < hi_v) ? *reinterpret_cast<const uint4*>(x + i + u * STEP)
                                         : make_uint4(ninf, ninf, ninf, ninf);
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          float f[2 * VEC];
#pragma unroll
          for (int u = 0; u < 2; ++u) {
            const T* e = reinterpret_cast<const T*>(&raw[2 * h + u]);
#pragma unroll
            for (int j = 0; j < VEC; ++j) f[u * VEC + j] = to_float(e[j]);
          }
          batch_add<2, VEC>(acc, f, i + 2 * h * STEP, STEP);
        }
      }
      for (int i = hi_v + threadIdx.x; i < hi; i += SAMPLE_THREADS) acc_add(acc, to_float(x[i]), i);
    } else {
      for (int i = lo + threadIdx.x; i < hi; i += SAMPLE_THREADS) acc_add(acc, to_float(x[i]), i);
    }
  }
  // CTA reduction
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    Acc b;
    b.m = __shfl_xor_sync(0xffffffffu, acc.m, o);
    b.s = __shfl_xor_sync(0xffffffffu, acc.s, o);
    b.idx = __shfl_xor_sync(0xffffffffu, acc.idx, o);
    acc = acc_merge(acc, b);
  }
  if ((threadIdx.x & 31) == 0) warp_acc[threadIdx.x >> 5] = acc;
  __syncthreads();
  __shared__ int is_last;
  if (threadIdx.x == 0) {
    Acc t = warp_acc[0];
    for (int w = 1; w < SAMPLE_THREADS / 32; ++w) t = acc_merge(t, warp_acc[w]);
    float* p = a.part + ((size_t)r * a.splits + sp) * 4;
    p[0] = t.m; p[1] = t.s; p[2] = __int_as_float(t.idx);
    __threadfence();
    const int old = atomicAdd(a.counters + r, 1);
    is_last = old == a.splits - 1;
    if (is_last) {
      a.counters[r] = 0;
      __threadfence();   // the other slices' partial results are visible from here on
    }
  }
  __syncthreads();
  if (!is_last || threadIdx.x >= 32) return;
  // The last CTA of the row to arrive: its first warp combines the slices, lane l slices l and l + 32,
  // then a fixed shuffle tree -- the result does not depend on who arrived when.
  const float* q = a.part + (size_t)r * a.splits * 4;
  Acc all{-INFINITY, 0.f, 0x7fffffff};
  for (int s2 = threadIdx.x; s2 < a.splits; s2 += 32) {
    const float4 v = __ldcg(reinterpret_cast<const float4*>(q + 4 * s2));
    all = acc_merge(all, Acc{v.x, v.y, __float_as_int(v.z)});
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    Acc b;
    b.m = __shfl_xor_sync(0xffffffffu, all.m, o);
    b.s = __shfl_xor_sync(0xffffffffu, all.s, o);
    b.idx = __shfl_xor_sync(0xffffffffu, all.idx, o);
    all = acc_merge(all, b);
  }
  if (threadIdx.x != 0) return;
  if (bad) {
    a.token[r] = -1; a.conf[r] = 0.f;
    if (a.lse) a.lse[r] = 0.f;
    if (atomicCAS(a.status, 0, (int)LACACHE_ERR_INVALID_ARG) == 0) { a.status[1] = LOC_SAMPLE_ROW; a.status[2] = r; a.status[3] = row; }
  } else {
    a.token[r] = all.idx;
    a.conf[r] = 1.f / all.s;                       // exp(x_max - x_max) / sum
    if (a.lse) a.lse[r] = all.m + log2f(all.s) * LN2F;
  }
}

}  // namespace

cudaError_t sample_rows(const SampleArgs& a, cudaStream_t s) {
  if (a.n_rows == 0) return cudaSuccess;
  dim3 grid(a.splits, a.n_rows);
  if (a.dtype == LACACHE_DTYPE_BF16) sample_rows_kernel<__nv_bfloat16><<<grid, SAMPLE_THREADS, 0, s>>>(a);
  else sample_rows_kernel<float><<<grid, SAMPLE_THREADS, 0, s>>>(a);
  return cudaGetLastError();
}

}  // namespace lacache
