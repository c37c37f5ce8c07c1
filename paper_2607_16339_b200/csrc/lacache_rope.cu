// RoPE-on-write (Eq. 1, Sec. 3.3.2) and the export kernels.
//
// rope_write rotates q and k at each token's position, copies v, and stores
// the result head-major in the engine's storage format:
//   SIMT engine    : fp32 planes.
//   tcgen05 engine : rotated q,k as two bf16 planes hi = bf16(x),
//                    lo = bf16(x - hi) (so hi + lo carries 16 significand
//                    bits into the tensor-core score product); v as fp16.
// The same kernel serves the build (all T tokens) and the step (only the
// block's L_b tokens per sequence, scattered to their cache slots).
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "lacache_internal.h"
#include "lacache_rope_math.h"

namespace lacache {
namespace {

__device__ __forceinline__ void store8_f32(void* plane, size_t off, const float (&y)[8]) {
  float4* p = reinterpret_cast<float4*>(reinterpret_cast<float*>(plane) + off);
  p[0] = make_float4(y[0], y[1], y[2], y[3]);
  p[1] = make_float4(y[4], y[5], y[6], y[7]);
}

__device__ __forceinline__ void store8_split(void* hi_plane, void* lo_plane, size_t off,
                                             const float (&y)[8], bool f16) {
  if (f16) {   // one fp16 plane: the rotated value rounded once to fp16
    *reinterpret_cast<uint4*>(reinterpret_cast<__half*>(hi_plane) + off) = rope_half8(y);
    return;
  }
  uint4 uh, ul;
  rope_split8(y, uh, ul);
  *reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(hi_plane) + off) = uh;
  // (plain operands keep the hi plane alone: the rotated value rounded once to bf16)
  if (lo_plane) *reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(lo_plane) + off) = ul;
}

__device__ __forceinline__ void store8_f16(void* plane, size_t off, const float (&y)[8]) {
  *reinterpret_cast<uint4*>(reinterpret_cast<__half*>(plane) + off) = rope_half8(y);
}

// One thread: 8 features c0..c0+7 of the first half and their partners at
// c0 + d/2 of one (source row, head slot).  Head slots: [0,Hq) q heads,
// [Hq,Hq+Hkv) k heads, [Hq+Hkv,Hq+2Hkv) v heads.
template <bool TC>
__global__ void __launch_bounds__(256) rope_write_kernel(Geometry g, RopeArgs a) {
  // the attention kernel that follows may be launched programmatically
  // dependent: let it start its prologue now (it waits for this grid's writes
  // before it touches them)
  // (when the kernel before this one writes this kernel's inputs, they are complete only after the
  // wait, and the attention kernel, which also reads them early, must not start before that)
  if (a.pdl == 2) asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int chunks = g.d / 16;
  const int slots = g.Hq + 2 * g.Hkv;
  const long long total = (long long)a.n_src_rows * slots * chunks;
  long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= total) return;
  int chunk = (int)(idx % chunks);
  long long t = idx / chunks;
  int slot = (int)(t % slots);
  int r = (int)(t / slots);
  int tok = a.row_tok ? a.row_tok[r] : (a.blk_start ? a.blk_start[r / a.block_len] + r % a.block_len : r);
  const int half = g.d / 2;
  const int c0 = chunk * 8;

  const void* src;
  int H, h;
  int which;  // 0 q, 1 k, 2 v
  if (slot < g.Hq) { src = a.q; H = g.Hq; h = slot; which = 0; }
  else if (slot < g.Hq + g.Hkv) { src = a.k; H = g.Hkv; h = slot - g.Hq; which = 1; }
  else { src = a.v; H = g.Hkv; h = slot - g.Hq - g.Hkv; which = 2; }

  float x1[8], x2[8], y1[8], y2[8];
  size_t soff = ((size_t)r * H + h) * g.d;
  rope_load8(src, soff + c0, a.in_dtype == LACACHE_DTYPE_BF16, x1);
  rope_load8(src, soff + c0 + half, a.in_dtype == LACACHE_DTYPE_BF16, x2);
  if (which < 2) {
    const float4 *cp, *sp;
    if (a.row_cos) {
      cp = reinterpret_cast<const float4*>(a.row_cos + (size_t)r * half + c0);
      sp = reinterpret_cast<const float4*>(a.row_sin + (size_t)r * half + c0);
    } else {
      int pos = a.pos_of_tok[tok];
      cp = reinterpret_cast<const float4*>(a.cos_tab + (size_t)pos * half + c0);
      sp = reinterpret_cast<const float4*>(a.sin_tab + (size_t)pos * half + c0);
    }
    float4 ca = cp[0], cb = cp[1], sa = sp[0], sb = sp[1];
    float cs[8] = {ca.x, ca.y, ca.z, ca.w, cb.x, cb.y, cb.z, cb.w};
    float sn[8] = {sa.x, sa.y, sa.z, sa.w, sb.x, sb.y, sb.z, sb.w};
    rope_rotate8(x1, x2, cs, sn, y1, y2);
  } else {
#pragma unroll
    for (int i = 0; i < 8; ++i) { y1[i] = x1[i]; y2[i] = x2[i]; }
  }
  // Everything above read only this call's inputs and constant tables.  The stores below overwrite
  // cache rows that the previous step's attention kernel may still be reading when this kernel was
  // launched programmatically dependent on it: wait for that grid first (returns at once otherwise).
  asm volatile("griddepcontrol.wait;" ::: "memory");
  size_t doff = ((size_t)h * g.Tp + tok) * g.d;
  if (TC) {
    // tcgen05 storage: [head][feature half][Tp][64] (d = 128), each half of a row one 128-byte line
    const size_t o1 = ((size_t)(2 * h) * g.Tp + tok) * 64 + c0;
    const size_t o2 = ((size_t)(2 * h + 1) * g.Tp + tok) * 64 + c0;
    if (which == 0) {
      store8_split(a.dst.q_hi, a.dst.q_lo, o1, y1, g.op_f16 != 0);
      store8_split(a.dst.q_hi, a.dst.q_lo, o2, y2, g.op_f16 != 0);
    } else if (which == 1) {
      store8_split(a.dst.k_hi, a.dst.k_lo, o1, y1, g.op_f16 != 0);
      store8_split(a.dst.k_hi, a.dst.k_lo, o2, y2, g.op_f16 != 0);
    } else {
      store8_f16(a.dst.v, o1, y1);
      store8_f16(a.dst.v, o2, y2);
    }
  } else {
    void* plane = which == 0 ? a.dst.q_hi : (which == 1 ? a.dst.k_hi : a.dst.v);
    store8_f32(plane, doff + c0, y1);
    store8_f32(plane, doff + c0 + half, y2);
  }
}

// Export kernels: head-major storage -> token-major fp32.
template <bool TC>
__device__ __forceinline__ float read_rot(const void* hi, const void* lo, size_t off, bool f16) {
  if (TC && f16) return __half2float(reinterpret_cast<const __half*>(hi)[off]);
  if (TC) {
    return __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(hi)[off]) +
           (lo ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(lo)[off]) : 0.f);
  }
  return reinterpret_cast<const float*>(hi)[off];
}

template <bool TC>
__global__ void __launch_bounds__(256) export_kernel(Geometry g, ExportArgs a) {
  long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  long long nq = (long long)g.T * g.Hq * g.d;
  if (idx >= nq) return;
  int c = (int)(idx % g.d);
  long long t = idx / g.d;
  int h = (int)(t % g.Hq);
  int tok = (int)(t / g.Hq);
  const size_t srow = ((size_t)h * g.Tp + tok) * g.d + c;   // state: [head][Tp][d]
  // rotated planes: the tcgen05 engine stores [head][feature half][Tp][64]
  const size_t src = TC ? ((size_t)(2 * h + c / 64) * g.Tp + tok) * 64 + c % 64 : srow;
  const float LN2 = 0.69314718055994530942f;
  if (a.o) a.o[idx] = a.st.o[srow];
  if (c == 0) {
    if (a.m) a.m[(size_t)tok * g.Hq + h] = a.st.m[(size_t)h * g.Tp + tok] * LN2;
    if (a.l) a.l[(size_t)tok * g.Hq + h] = a.st.l[(size_t)h * g.Tp + tok];
  }
  if (a.q_rot) a.q_rot[idx] = read_rot<TC>(a.rot.q_hi, a.rot.q_lo, src, g.op_f16 != 0);
  if (h < g.Hkv) {
    size_t dst = ((size_t)tok * g.Hkv + h) * g.d + c;
    if (a.k_rot) a.k_rot[dst] = read_rot<TC>(a.rot.k_hi, a.rot.k_lo, src, g.op_f16 != 0);
    if (a.v) {
      a.v[dst] = TC ? __half2float(reinterpret_cast<const __half*>(a.rot.v)[src])
                    : reinterpret_cast<const float*>(a.rot.v)[src];
    }
  }
}

// Partial states of the key chunks of block rows -> the rows' state (Eq. 2-6 merge): thread = 16 bytes of
// one row of one head; every load of the (at most eight at a time) chunks is issued before any is used.
__global__ void __launch_bounds__(256) merge_chunk_states_kernel(Geometry g, ChunkMergeArgs a) {
  // launched programmatically dependent on the kernel that writes the partial states: the launch itself and
  // the start of the kernel after this one overlap their neighbours; nothing is read before that kernel is complete
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int i = blockIdx.x * 256 + threadIdx.x;
  if (i >= g.block_len * 32) return;
  const int rr = i >> 5, ch = i & 31, h = blockIdx.y, b = blockIdx.z;
  const int row0 = a.tab[2 * b], n = a.tab[2 * b + 1];
  const size_t pbase = ((size_t)b * g.Hq + h) * a.max_chunks;
  float M = -INFINITY, L = 0.f;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int c0 = 0; c0 < n; c0 += 8) {
    float mv[8], lv[8];
    float4 v[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      if (c0 + k < n) {
        const size_t pr = (pbase + c0 + k) * g.block_len + rr;
        mv[k] = __ldcg(a.part_m + pr);
        lv[k] = __ldcg(a.part_l + pr);
        v[k] = __ldcg(reinterpret_cast<const float4*>(a.part_o + pr * g.d) + ch);
      } else {
        mv[k] = -INFINITY; lv[k] = 0.f; v[k] = make_float4(0.f, 0.f, 0.f, 0.f);
      }
    }
    float Mn = M;
#pragma unroll
    for (int k = 0; k < 8; ++k) Mn = fmaxf(Mn, mv[k]);
    const float w0 = (M == -INFINITY) ? 0.f : exp2f(M - Mn);
    L *= w0; acc.x *= w0; acc.y *= w0; acc.z *= w0; acc.w *= w0;
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      const float w = (mv[k] == -INFINITY) ? 0.f : exp2f(mv[k] - Mn);
      L = fmaf(lv[k], w, L);
      acc.x = fmaf(v[k].x, w, acc.x);
      acc.y = fmaf(v[k].y, w, acc.y);
      acc.z = fmaf(v[k].z, w, acc.z);
      acc.w = fmaf(v[k].w, w, acc.w);
    }
    M = Mn;
  }
  const size_t srow = (size_t)h * g.Tp + row0 + rr;
  *reinterpret_cast<float4*>(a.st.o + srow * g.d + ch * 4) = acc;
  if (ch == 0) { a.st.m[srow] = M; a.st.l[srow] = L; }
}

}  // namespace

cudaError_t merge_chunk_states(const Geometry& g, const ChunkMergeArgs& a, cudaStream_t s) {
  // (head_dim 128: 32 sixteen-byte columns per row, the only shape the tcgen05 engine serves)
  dim3 grid((unsigned)((g.block_len * 32 + 255) / 256), (unsigned)g.Hq, (unsigned)g.B);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = dim3(256);
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = a.no_pdl ? 0 : 1;
  return cudaLaunchKernelEx(&cfg, merge_chunk_states_kernel, g, a);
}

cudaError_t rope_write(const Geometry& g, const RopeArgs& a, int engine, cudaStream_t s) {
  long long total = (long long)a.n_src_rows * (g.Hq + 2 * g.Hkv) * (g.d / 16);
  if (total == 0) return cudaSuccess;
  unsigned blocks = (unsigned)((total + 255) / 256);
  if (engine == LACACHE_ENGINE_TCGEN05) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(blocks);
    cfg.blockDim = dim3(256);
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = (a.pdl && !a.no_pdl) ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, rope_write_kernel<true>, g, a);
  }
  rope_write_kernel<false><<<blocks, 256, 0, s>>>(g, a);
  return cudaGetLastError();
}

cudaError_t export_buffers(const Geometry& g, const ExportArgs& a, int engine, cudaStream_t s) {
  long long total = (long long)g.T * g.Hq * g.d;
  unsigned blocks = (unsigned)((total + 255) / 256);
  if (engine == LACACHE_ENGINE_TCGEN05)
    export_kernel<true><<<blocks, 256, 0, s>>>(g, a);
  else
    export_kernel<false><<<blocks, 256, 0, s>>>(g, a);
  return cudaGetLastError();
}

}  // namespace lacache
