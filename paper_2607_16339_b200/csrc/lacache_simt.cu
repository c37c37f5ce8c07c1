// CUDA-core fp32 attention kernels (the fp32 dtype path, and any shape the
// tcgen05 path does not cover).  One generic kernel runs every mode:
//   build : fixed queries x fixed keys            -> cached (m, l, O~)
//   step  : fixed queries x block keys, starting from the cached state
//           (Algorithm 1 reuse pass); block queries x all keys
//   full  : all queries x all keys (no cache)
// following the online-softmax recurrence of Eq. 2-6 with key tiles of 32.
//
// Mapping: a CTA owns 32 query rows of one (sequence, q head); each of its 8
// warps owns 4 rows.  Per key tile, lane j holds the score of key j for the
// warp's 4 rows (dot product over d from shared memory), row max / sum are
// warp shuffles, and for P.V lane c owns output features c, c+32, ...
#include <cuda_bf16.h>

#include "lacache_internal.h"

namespace lacache {
namespace {

constexpr int KT = 32;    // keys per tile
constexpr int RPW = 4;    // rows per warp
constexpr int WARPS = 8;

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

template <int D>
__global__ void __launch_bounds__(WARPS * 32) simt_attn_kernel(Geometry g, AttnArgs a) {
  constexpr int DPL = D / 32;  // output features per lane
  extern __shared__ float sm[];
  float* Qs = sm;                         // [32][D]
  float* Ks = Qs + SIMT_ROWS * D;         // [KT][D+1]
  float* Vs = Ks + KT * (D + 1);          // [KT][D]

  const WorkItem it = a.items[blockIdx.x];
  const int h = blockIdx.y;
  const int kh = h / g.group;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int seq_start = a.cu[it.seq], seq_end = a.cu[it.seq + 1];
  const int bs = a.blk_start ? a.blk_start[it.seq] : 0;
  const int be = bs + g.block_len;

  int k0, k1, x0 = 0, x1 = 0;
  bool from_state = false, to_state = false;
  if (a.mode == MODE_BUILD) {
    k0 = seq_start; k1 = seq_end; x0 = bs; x1 = be; to_state = true;
  } else if (a.mode == MODE_STEP && it.kind == ITEM_ROWS) {
    k0 = bs; k1 = be; from_state = true;
  } else {
    k0 = seq_start; k1 = seq_end;
  }

  const float* qr = reinterpret_cast<const float*>(a.rot.q_hi) + (size_t)h * g.Tp * D;
  const float* kr = reinterpret_cast<const float*>(a.rot.k_hi) + (size_t)kh * g.Tp * D;
  const float* vr = reinterpret_cast<const float*>(a.rot.v) + (size_t)kh * g.Tp * D;

  // stage the query rows
  for (int i = threadIdx.x; i < SIMT_ROWS * (D / 4); i += blockDim.x) {
    int r = i / (D / 4), c4 = i % (D / 4);
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (r < it.nrows) v = *reinterpret_cast<const float4*>(qr + (size_t)(it.row0 + r) * D + c4 * 4);
    *reinterpret_cast<float4*>(Qs + r * D + c4 * 4) = v;
  }

  float m[RPW], l[RPW], o[RPW][DPL];
#pragma unroll
  for (int i = 0; i < RPW; ++i) {
    int r = warp * RPW + i;
    m[i] = -INFINITY;
    l[i] = 0.f;
#pragma unroll
    for (int t = 0; t < DPL; ++t) o[i][t] = 0.f;
    if (from_state && r < it.nrows) {
      size_t row = (size_t)h * g.Tp + it.row0 + r;
      m[i] = a.st.m[row];
      l[i] = a.st.l[row];
#pragma unroll
      for (int t = 0; t < DPL; ++t) o[i][t] = a.st.o[row * D + lane + 32 * t];
    }
  }

  for (int kt = k0; kt < k1; kt += KT) {
    // a tile entirely inside the excluded range contributes nothing
    if (kt >= x0 && min(kt + KT, k1) <= x1 && x1 > x0) continue;
    __syncthreads();
    for (int i = threadIdx.x; i < KT * (D / 4); i += blockDim.x) {
      int r = i / (D / 4), c4 = i % (D / 4);
      float4 kv = make_float4(0.f, 0.f, 0.f, 0.f), vv = kv;
      if (kt + r < k1) {
        kv = *reinterpret_cast<const float4*>(kr + (size_t)(kt + r) * D + c4 * 4);
        vv = *reinterpret_cast<const float4*>(vr + (size_t)(kt + r) * D + c4 * 4);
      }
      float* kd = Ks + r * (D + 1) + c4 * 4;
      kd[0] = kv.x; kd[1] = kv.y; kd[2] = kv.z; kd[3] = kv.w;
      *reinterpret_cast<float4*>(Vs + r * D + c4 * 4) = vv;
    }
    __syncthreads();

    const int key = kt + lane;
    const bool valid = key < k1 && !(key >= x0 && key < x1);
    float s[RPW];
#pragma unroll
    for (int i = 0; i < RPW; ++i) s[i] = 0.f;
    const float* krow = Ks + lane * (D + 1);
    const float* qw = Qs + warp * RPW * D;
#pragma unroll 8
    for (int c = 0; c < D; ++c) {
      float kv = krow[c];
#pragma unroll
      for (int i = 0; i < RPW; ++i) s[i] = fmaf(qw[i * D + c], kv, s[i]);
    }
#pragma unroll
    for (int i = 0; i < RPW; ++i) {
      float sv = valid ? s[i] * g.scale_log2 : -INFINITY;
      float m_new = fmaxf(m[i], warp_max(sv));
      if (m_new == -INFINITY) continue;  // nothing seen yet (warp-uniform)
      float alpha = (m[i] == -INFINITY) ? 0.f : exp2f(m[i] - m_new);
      float p = valid ? exp2f(sv - m_new) : 0.f;
      l[i] = l[i] * alpha + warp_sum(p);
      m[i] = m_new;
#pragma unroll
      for (int t = 0; t < DPL; ++t) o[i][t] *= alpha;
#pragma unroll 8
      for (int j = 0; j < KT; ++j) {
        float pj = __shfl_sync(0xffffffffu, p, j);
#pragma unroll
        for (int t = 0; t < DPL; ++t) o[i][t] = fmaf(pj, Vs[j * D + lane + 32 * t], o[i][t]);
      }
    }
  }

  const float LN2 = 0.69314718055994530942f;
#pragma unroll
  for (int i = 0; i < RPW; ++i) {
    int r = warp * RPW + i;
    if (r >= it.nrows) continue;
    int tok = it.row0 + r;
    if (to_state) {
      size_t row = (size_t)h * g.Tp + tok;
      if (lane == 0) { a.st.m[row] = m[i]; a.st.l[row] = l[i]; }
#pragma unroll
      for (int t = 0; t < DPL; ++t) a.st.o[row * D + lane + 32 * t] = o[i][t];
    } else {
      float inv = 1.f / l[i];
      size_t row = (size_t)tok * g.Hq + h;
      if (a.out_bf16) {
        __nv_bfloat16* ob = reinterpret_cast<__nv_bfloat16*>(a.out);
#pragma unroll
        for (int t = 0; t < DPL; ++t) ob[row * D + lane + 32 * t] = __float2bfloat16_rn(o[i][t] * inv);
      } else {
#pragma unroll
        for (int t = 0; t < DPL; ++t) a.out[row * D + lane + 32 * t] = o[i][t] * inv;
      }
      if (a.lse && lane == 0) a.lse[row] = (m[i] + log2f(l[i])) * LN2;
    }
  }
}

template <int D>
constexpr size_t simt_smem() {
  return sizeof(float) * (SIMT_ROWS * D + KT * (D + 1) + KT * D);
}

}  // namespace

cudaError_t simt_prepare() {
  cudaError_t e = cudaFuncSetAttribute(simt_attn_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)simt_smem<128>());
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(simt_attn_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              (int)simt_smem<64>());
}

cudaError_t simt_attention(const Geometry& g, const AttnArgs& a, cudaStream_t s) {
  if (a.n_items == 0) return cudaSuccess;
  dim3 grid(a.n_items, g.Hq);
  if (g.d == 128)
    simt_attn_kernel<128><<<grid, WARPS * 32, simt_smem<128>(), s>>>(g, a);
  else
    simt_attn_kernel<64><<<grid, WARPS * 32, simt_smem<64>(), s>>>(g, a);
  return cudaGetLastError();
}

}  // namespace lacache
