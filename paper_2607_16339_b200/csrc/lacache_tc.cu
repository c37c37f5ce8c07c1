// tcgen05 attention kernels for sm_100a (bf16 inputs, head_dim 128).
//
// One CTA owns a tile of 128 query rows of one (sequence, q head) and streams
// key tiles of 64 keys through the online-softmax recurrence of Eq. 2-6:
//   S  = Q' K'^T      tcgen05.mma kind::f16 (bf16 operands from shared memory,
//                     fp32 accumulator in TMEM).  Rotated Q' and K' are stored
//                     as hi + lo bf16 planes and the product is formed as
//                     hi.hi + hi.lo + lo.hi so the scores carry ~16 significand
//                     bits of each operand.
//   P~ = exp2(S c - m) computed by 128 threads, one TMEM lane (= query row)
//                     each, with an INTEGER reference exponent m (so every
//                     rescale factor is an exact power of two), rounded to
//                     fp16 and written back to TMEM.
//   O~ += P~ V        tcgen05.mma with A = P~ read from TMEM and B = V (fp16,
//                     MN-major) from shared memory.
// Q, K and V tiles are staged by TMA (128-byte swizzle) and tracked by
// mbarriers; every wait is bounded and reports through the status word.
//
// The same kernel runs all modes (what the key range is, where the state
// starts and where the result goes):
//   build : rows in U, keys in U                    -> cached (m, l, O~)
//   step  : rows in U start from the cache, keys = the block        -> out
//           rows in C, keys = one chunk of all keys -> partial state; the
//           last chunk to arrive merges the partials                -> out
//   full  : all rows, all keys                                      -> out
#include <cuda.h>
#include <cuda_fp16.h>
#include <stdio.h>

#include "lacache_internal.h"

namespace lacache {

struct TcMaps {
  alignas(64) CUtensorMap q_hi;
  alignas(64) CUtensorMap q_lo;
  alignas(64) CUtensorMap k_hi;
  alignas(64) CUtensorMap k_lo;
  alignas(64) CUtensorMap v;
};

namespace {

constexpr int D = 128;
constexpr int BM = TC_ROWS;   // 128 query rows
constexpr int BN = TC_KEYS;   // 64 keys
constexpr int THREADS = 128;

// shared memory map (bytes, from a 1024-aligned base)
constexpr uint32_t SM_QHI = 0;                    // 2 boxes [128 rows][64 cols] bf16
constexpr uint32_t SM_QLO = SM_QHI + 32768;
constexpr uint32_t SM_KHI = SM_QLO + 32768;       // 2 boxes [64 rows][64 cols] bf16
constexpr uint32_t SM_KLO = SM_KHI + 16384;
constexpr uint32_t SM_V = SM_KLO + 16384;         // 2 boxes [64 keys][64 cols] fp16
constexpr uint32_t SM_BAR = SM_V + 16384;         // mbarriers + small words
constexpr uint32_t SM_TOTAL = SM_BAR + 128;
constexpr uint32_t Q_BOX_BYTES = 128 * 128;       // 128 rows x 128 B
constexpr uint32_t K_BOX_BYTES = 64 * 128;

// TMEM columns (fp32 words per lane)
constexpr uint32_t TM_S = 0;      // 64 columns: scores
constexpr uint32_t TM_P = 64;     // 32 columns: 64 fp16 probabilities, packed
constexpr uint32_t TM_O = 128;    // 128 columns: P.V of the current tile
constexpr uint32_t TM_COLS = 256;

// barrier slots
enum { BAR_Q = 0, BAR_K, BAR_V, BAR_S, BAR_O, BAR_SYNC, BAR_DONE, N_BARS };

constexpr long long WAIT_CYCLES = 3000000000ll;  // ~1.5 s at 2 GHz

// ---- PTX wrappers ----------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0,
                                            int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem]
__device__ __forceinline__ void mma_ss(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                       uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem]
__device__ __forceinline__ void mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc,
                                       uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
        "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// shared-memory matrix descriptor, 128-byte swizzle, sm_100 version field
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  return (uint64_t)((addr >> 4) & 0x3FFFu) | ((uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16) |
         ((uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32) | (1ull << 46) | (2ull << 61);
}
// instruction descriptor for kind::f16: fp32 accumulate, M x N
constexpr uint32_t idesc_f16(uint32_t ab_format, uint32_t b_mn_major, uint32_t M, uint32_t N) {
  return (1u << 4) | (ab_format << 7) | (ab_format << 10) | (b_mn_major << 16) | ((N >> 3) << 17) |
         ((M >> 4) << 24);
}
constexpr uint32_t IDESC_S = idesc_f16(1u /*bf16*/, 0u, BM, BN);
constexpr uint32_t IDESC_PV = idesc_f16(0u /*f16*/, 1u, BM, D);

struct Shared {
  uint32_t base;       // shared-space address of the 1024-aligned region
  volatile int* abort_flag;
  int32_t* status;
};

// Bounded wait: false if the barrier did not complete in time or another
// thread of the CTA already gave up.
__device__ __forceinline__ bool wait_bar(const Shared& sh, int slot, uint32_t parity, int loc) {
  uint32_t bar = sh.base + SM_BAR + 8u * slot;
  if (mbar_try(bar, parity)) return true;
  long long t0 = clock64();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 64; ++i)
      if (mbar_try(bar, parity)) return true;
    if (*sh.abort_flag) return false;
    if (clock64() - t0 > WAIT_CYCLES) {
      *sh.abort_flag = 1;
      if (atomicCAS(sh.status, 0, (int)LACACHE_ERR_TIMEOUT) == 0) {
        sh.status[1] = loc;
        sh.status[2] = blockIdx.x;
        sh.status[3] = threadIdx.x;
      }
      return false;
    }
  }
}

__global__ void __launch_bounds__(THREADS, 2)
tc_attn_kernel(const __grid_constant__ TcMaps maps, const Geometry g, const AttnArgs a) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const int tid = threadIdx.x;
  const int warp = tid >> 5;
  Shared sh;
  sh.base = smem_u32(smem_raw);
  uint32_t* words = reinterpret_cast<uint32_t*>(smem_raw + SM_BAR + 8 * N_BARS);  // [0] tmem base, [1] abort, [2] last flag
  sh.abort_flag = reinterpret_cast<volatile int*>(words + 1);
  sh.status = a.status;
  if ((sh.base & 1023u) != 0) {  // swizzled tiles need a 1024-byte aligned base
    if (tid == 0 && atomicCAS(a.status, 0, (int)LACACHE_ERR_CUDA) == 0) a.status[1] = LOC_SMEM_ALIGN;
    return;
  }
  auto bar = [&](int slot) { return sh.base + SM_BAR + 8u * slot; };

  // ---- work item ----
  const WorkItem it = a.items[blockIdx.x];
  const int h = blockIdx.y;
  const int kh = h / g.group;
  const int seq_start = a.cu[it.seq], seq_end = a.cu[it.seq + 1];
  const int bs = a.blk_start ? a.blk_start[it.seq] : 0;
  const int be = bs + g.block_len;
  int key_base, t0, t1, k0, k1, x0 = 0, x1 = 0;
  bool from_state = false;
  const bool chunked = (a.mode == MODE_STEP && it.kind == ITEM_BLOCK_CHUNK);
  if (a.mode == MODE_BUILD) {
    key_base = seq_start; k0 = seq_start; k1 = seq_end; x0 = bs; x1 = be;
    t0 = 0; t1 = (seq_end - seq_start + BN - 1) / BN;
  } else if (a.mode == MODE_STEP && !chunked) {
    key_base = bs; k0 = bs; k1 = be; from_state = true;
    t0 = 0; t1 = (g.block_len + BN - 1) / BN;
  } else {
    key_base = seq_start; k0 = seq_start; k1 = seq_end;
    t0 = 0; t1 = (seq_end - seq_start + BN - 1) / BN;
    if (chunked) { t0 = it.kt0; t1 = it.kt1; }
  }
  // a key tile that lies entirely inside the excluded range is skipped
  auto tile_skipped = [&](int t) {
    int lo = key_base + t * BN, hi = min(lo + BN, k1);
    return x1 > x0 && lo >= x0 && hi <= x1;
  };
  auto next_tile = [&](int t) {
    while (t < t1 && tile_skipped(t)) ++t;
    return t;
  };

  // ---- setup: barriers, TMEM ----
  if (tid == 0) {
    mbar_init(bar(BAR_Q), 1);
    mbar_init(bar(BAR_K), 1);
    mbar_init(bar(BAR_V), 1);
    mbar_init(bar(BAR_S), 1);
    mbar_init(bar(BAR_O), 1);
    mbar_init(bar(BAR_SYNC), THREADS);
    mbar_init(bar(BAR_DONE), THREADS);
    words[1] = 0;
    words[2] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncwarp();
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(words)),
                 "r"(TM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = words[0];
  const uint32_t tlane = tmem + ((uint32_t)(warp * 32) << 16);  // this warp's 32 lanes

  uint32_t ph_q = 0, ph_k = 0, ph_v = 0, ph_s = 0, ph_o = 0, ph_sync = 0;
  bool ok = true;

  int t = next_tile(t0);
  if (tid == 0) {
    mbar_expect_tx(bar(BAR_Q), 4 * Q_BOX_BYTES);
    tma_load_3d(sh.base + SM_QHI, &maps.q_hi, bar(BAR_Q), 0, it.row0, h);
    tma_load_3d(sh.base + SM_QHI + Q_BOX_BYTES, &maps.q_hi, bar(BAR_Q), 64, it.row0, h);
    tma_load_3d(sh.base + SM_QLO, &maps.q_lo, bar(BAR_Q), 0, it.row0, h);
    tma_load_3d(sh.base + SM_QLO + Q_BOX_BYTES, &maps.q_lo, bar(BAR_Q), 64, it.row0, h);
    if (t < t1) {
      int krow = key_base + t * BN;
      mbar_expect_tx(bar(BAR_K), 4 * K_BOX_BYTES);
      tma_load_3d(sh.base + SM_KHI, &maps.k_hi, bar(BAR_K), 0, krow, kh);
      tma_load_3d(sh.base + SM_KHI + K_BOX_BYTES, &maps.k_hi, bar(BAR_K), 64, krow, kh);
      tma_load_3d(sh.base + SM_KLO, &maps.k_lo, bar(BAR_K), 0, krow, kh);
      tma_load_3d(sh.base + SM_KLO + K_BOX_BYTES, &maps.k_lo, bar(BAR_K), 64, krow, kh);
      mbar_expect_tx(bar(BAR_V), 2 * K_BOX_BYTES);
      tma_load_3d(sh.base + SM_V, &maps.v, bar(BAR_V), 0, krow, kh);
      tma_load_3d(sh.base + SM_V + K_BOX_BYTES, &maps.v, bar(BAR_V), 64, krow, kh);
    }
  }
  __syncwarp();

  // ---- per-row state: thread tid owns query row it.row0 + tid ----
  const int row = it.row0 + tid;
  const bool row_valid = tid < it.nrows;
  float m_run = -INFINITY, l_run = 0.f;
  float o_acc[D];
#pragma unroll
  for (int c = 0; c < D; ++c) o_acc[c] = 0.f;
  if (from_state && row_valid) {
    size_t srow = (size_t)h * g.Tp + row;
    m_run = a.st.m[srow];
    l_run = a.st.l[srow];
    const float4* src = reinterpret_cast<const float4*>(a.st.o + srow * D);
#pragma unroll
    for (int c = 0; c < D / 4; ++c) {
      float4 v = src[c];
      o_acc[4 * c] = v.x; o_acc[4 * c + 1] = v.y; o_acc[4 * c + 2] = v.z; o_acc[4 * c + 3] = v.w;
    }
  }

  if (tid == 0) ok = wait_bar(sh, BAR_Q, ph_q, LOC_WAIT_Q);  // always: no copy may outlive the CTA
  ph_q ^= 1;

  while (ok && t < t1) {
    const int tn = next_tile(t + 1);
    const int tile_lo = key_base + t * BN;
    // ---- S = Q' K'^T ----
    if (tid == 0) {
      ok = wait_bar(sh, BAR_K, ph_k, LOC_WAIT_K);
      if (ok) {
        tc_fence_after();
        uint32_t acc = 0;
#pragma unroll
        for (int term = 0; term < 3; ++term) {
          // hi.hi, hi.lo, lo.hi
          const uint32_t qa = sh.base + (term == 2 ? SM_QLO : SM_QHI);
          const uint32_t ka = sh.base + (term == 1 ? SM_KLO : SM_KHI);
#pragma unroll
          for (int ks = 0; ks < D / 16; ++ks) {
            uint32_t qoff = (ks >> 2) * Q_BOX_BYTES + (ks & 3) * 32;
            uint32_t koff = (ks >> 2) * K_BOX_BYTES + (ks & 3) * 32;
            mma_ss(tmem + TM_S, smem_desc(qa + qoff, 16, 1024), smem_desc(ka + koff, 16, 1024), IDESC_S, acc);
            acc = 1;
          }
        }
        tc_commit(bar(BAR_S));
      }
    }
    __syncwarp();
    ph_k ^= 1;
    if (!wait_bar(sh, BAR_S, ph_s, LOC_WAIT_S)) { ok = false; break; }
    ph_s ^= 1;
    tc_fence_after();
    if (tid == 0 && tn < t1) {  // the K buffers are free: prefetch the next tile's keys
      int krow = key_base + tn * BN;
      mbar_expect_tx(bar(BAR_K), 4 * K_BOX_BYTES);
      tma_load_3d(sh.base + SM_KHI, &maps.k_hi, bar(BAR_K), 0, krow, kh);
      tma_load_3d(sh.base + SM_KHI + K_BOX_BYTES, &maps.k_hi, bar(BAR_K), 64, krow, kh);
      tma_load_3d(sh.base + SM_KLO, &maps.k_lo, bar(BAR_K), 0, krow, kh);
      tma_load_3d(sh.base + SM_KLO + K_BOX_BYTES, &maps.k_lo, bar(BAR_K), 64, krow, kh);
    }
    __syncwarp();

    // ---- online softmax on this thread's row ----
    // column j of the tile is key tile_lo + j; valid keys: [k0,k1) minus [x0,x1)
    const int v_lo = max(k0 - tile_lo, 0), v_hi = min(k1 - tile_lo, BN);
    const int e_lo = x0 - tile_lo, e_hi = x1 - tile_lo;
    auto col_valid = [&](int j) { return j >= v_lo && j < v_hi && !(j >= e_lo && j < e_hi); };
    float mx = -INFINITY;
#pragma unroll
    for (int half = 0; half < 2; ++half) {
      uint32_t r[32];
      tmem_ld32(tlane + TM_S + 32 * half, r);
      tmem_ld_wait();
#pragma unroll
      for (int j = 0; j < 32; ++j)
        if (col_valid(32 * half + j)) mx = fmaxf(mx, __uint_as_float(r[j]));
    }
    // integer reference exponent (log2 units) so rescales are exact powers of two
    const float m_new = fmaxf(m_run, ceilf(mx * g.scale_log2));
    const float m_ref = (m_new == -INFINITY) ? 0.f : m_new;
    const float alpha = (m_run == -INFINITY) ? 0.f : ex2(m_run - m_new);
    float psum = 0.f;
#pragma unroll
    for (int half = 0; half < 2; ++half) {
      uint32_t r[32];
      tmem_ld32(tlane + TM_S + 32 * half, r);
      tmem_ld_wait();
      uint32_t pk[16];
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        int c = 32 * half + 2 * j;
        float p0 = col_valid(c) ? ex2(fmaf(__uint_as_float(r[2 * j]), g.scale_log2, -m_ref)) : 0.f;
        float p1 = col_valid(c + 1) ? ex2(fmaf(__uint_as_float(r[2 * j + 1]), g.scale_log2, -m_ref)) : 0.f;
        __half2 hp = __floats2half2_rn(p0, p1);
        float2 back = __half22float2(hp);
        psum += back.x + back.y;  // the normaliser sums exactly what the MMA multiplies
        pk[j] = *reinterpret_cast<uint32_t*>(&hp);
      }
      tmem_st16(tlane + TM_P + 16 * half, pk);
    }
    tmem_st_wait();
    l_run = l_run * alpha + psum;
    m_run = m_new;
    // every thread's P~ is in TMEM before the MMA reads it
    tc_fence_before();
    mbar_arrive(bar(BAR_SYNC));
    if (tid == 0) {
      ok = wait_bar(sh, BAR_SYNC, ph_sync, LOC_WAIT_S);
      if (ok) ok = wait_bar(sh, BAR_V, ph_v, LOC_WAIT_V);
      if (ok) {
        tc_fence_after();
#pragma unroll
        for (int ks = 0; ks < BN / 16; ++ks) {
          // B = V tile, MN-major: 64 features contiguous, next 64 at +8 KB (LBO),
          // groups of 8 keys 1 KB apart (SBO); 16 keys per MMA = 2 KB
          mma_ts(tmem + TM_O, tmem + TM_P + 8 * ks, smem_desc(sh.base + SM_V + ks * 2048, K_BOX_BYTES, 1024),
                 IDESC_PV, ks > 0 ? 1u : 0u);
        }
        tc_commit(bar(BAR_O));
      }
    }
    __syncwarp();
    ph_sync ^= 1;
    ph_v ^= 1;
    if (!wait_bar(sh, BAR_O, ph_o, LOC_WAIT_O)) { ok = false; break; }
    ph_o ^= 1;
    tc_fence_after();
    if (tid == 0 && tn < t1) {  // the V buffer is free
      int krow = key_base + tn * BN;
      mbar_expect_tx(bar(BAR_V), 2 * K_BOX_BYTES);
      tma_load_3d(sh.base + SM_V, &maps.v, bar(BAR_V), 0, krow, kh);
      tma_load_3d(sh.base + SM_V + K_BOX_BYTES, &maps.v, bar(BAR_V), 64, krow, kh);
    }
    __syncwarp();
    // ---- O~ = alpha O~ + P~ V ----
#pragma unroll
    for (int q4 = 0; q4 < 4; ++q4) {
      uint32_t r[32];
      tmem_ld32(tlane + TM_O + 32 * q4, r);
      tmem_ld_wait();
#pragma unroll
      for (int j = 0; j < 32; ++j) o_acc[32 * q4 + j] = fmaf(o_acc[32 * q4 + j], alpha, __uint_as_float(r[j]));
    }
    tc_fence_before();
    t = tn;
  }

  // ---- epilogue ----
  const float LN2 = 0.69314718055994530942f;
  if (ok && row_valid) {
    if (a.mode == MODE_BUILD) {
      size_t srow = (size_t)h * g.Tp + row;
      a.st.m[srow] = m_run;
      a.st.l[srow] = l_run;
      float4* dst = reinterpret_cast<float4*>(a.st.o + srow * D);
#pragma unroll
      for (int c = 0; c < D / 4; ++c)
        dst[c] = make_float4(o_acc[4 * c], o_acc[4 * c + 1], o_acc[4 * c + 2], o_acc[4 * c + 3]);
    } else if (!chunked || it.pad == 1) {
      const float inv = 1.f / l_run;
      size_t orow = (size_t)row * g.Hq + h;
      float4* dst = reinterpret_cast<float4*>(a.out + orow * D);
#pragma unroll
      for (int c = 0; c < D / 4; ++c)
        dst[c] = make_float4(o_acc[4 * c] * inv, o_acc[4 * c + 1] * inv, o_acc[4 * c + 2] * inv, o_acc[4 * c + 3] * inv);
      if (a.lse) a.lse[orow] = (m_run + log2f(l_run)) * LN2;
    } else {
      size_t prow = (((size_t)it.seq * g.Hq + h) * a.max_chunks + it.chunk) * g.block_len + tid;
      a.part_m[prow] = m_run;
      a.part_l[prow] = l_run;
      float4* dst = reinterpret_cast<float4*>(a.part_o + prow * D);
#pragma unroll
      for (int c = 0; c < D / 4; ++c)
        dst[c] = make_float4(o_acc[4 * c], o_acc[4 * c + 1], o_acc[4 * c + 2], o_acc[4 * c + 3]);
    }
  }
  if (chunked && it.pad > 1) {
    // the last chunk of this (sequence, head) to arrive merges all partials
    __threadfence();
    mbar_arrive(bar(BAR_SYNC));
    bool synced = wait_bar(sh, BAR_SYNC, ph_sync, LOC_WAIT_O);
    ph_sync ^= 1;
    if (synced && tid == 0) {
      int old = atomicAdd(&a.counters[it.seq * g.Hq + h], 1);
      int last = (old == it.pad - 1) ? 1 : 0;
      if (last) a.counters[it.seq * g.Hq + h] = 0;
      words[2] = last;
      __threadfence();
    }
    mbar_arrive(bar(BAR_SYNC));
    synced = synced && wait_bar(sh, BAR_SYNC, ph_sync, LOC_WAIT_O);
    ph_sync ^= 1;
    if (synced && ok && words[2] && row_valid) {
      __threadfence();
      size_t p0 = (((size_t)it.seq * g.Hq + h) * a.max_chunks) * g.block_len + tid;
      float M = -INFINITY;
      for (int c = 0; c < it.pad; ++c) M = fmaxf(M, __ldcg(a.part_m + p0 + (size_t)c * g.block_len));
      float L = 0.f;
#pragma unroll
      for (int c = 0; c < D; ++c) o_acc[c] = 0.f;
      for (int ch = 0; ch < it.pad; ++ch) {
        size_t pr = p0 + (size_t)ch * g.block_len;
        float mc = __ldcg(a.part_m + pr);
        if (mc == -INFINITY) continue;
        float w = ex2(mc - M);
        L = fmaf(__ldcg(a.part_l + pr), w, L);
        const float4* src = reinterpret_cast<const float4*>(a.part_o + pr * D);
#pragma unroll
        for (int c = 0; c < D / 4; ++c) {
          float4 v = __ldcg(src + c);
          o_acc[4 * c] = fmaf(v.x, w, o_acc[4 * c]);
          o_acc[4 * c + 1] = fmaf(v.y, w, o_acc[4 * c + 1]);
          o_acc[4 * c + 2] = fmaf(v.z, w, o_acc[4 * c + 2]);
          o_acc[4 * c + 3] = fmaf(v.w, w, o_acc[4 * c + 3]);
        }
      }
      const float inv = 1.f / L;
      size_t orow = (size_t)row * g.Hq + h;
      float4* dst = reinterpret_cast<float4*>(a.out + orow * D);
#pragma unroll
      for (int c = 0; c < D / 4; ++c)
        dst[c] = make_float4(o_acc[4 * c] * inv, o_acc[4 * c + 1] * inv, o_acc[4 * c + 2] * inv, o_acc[4 * c + 3] * inv);
      if (a.lse) a.lse[orow] = (M + log2f(L)) * LN2;
    }
  }

  // ---- teardown: free TMEM once every thread is past its last TMEM access ----
  tc_fence_before();
  mbar_arrive(bar(BAR_DONE));
  if (warp == 0) {
    wait_bar(sh, BAR_DONE, 0, LOC_WAIT_O);
    __syncwarp();
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TM_COLS) : "memory");
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode() {
  static EncodeTiledFn fn = nullptr;
  if (fn) return fn;
  void* p = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess ||
      qres != cudaDriverEntryPointSuccess)
    return nullptr;
  fn = reinterpret_cast<EncodeTiledFn>(p);
  return fn;
}

bool make_plane_map(CUtensorMap* m, void* base, int H, int Tp, int box_rows, bool fp16, char* err, int errlen) {
  EncodeTiledFn enc = get_encode();
  if (!enc) { snprintf(err, errlen, "cuTensorMapEncodeTiled entry point not found"); return false; }
  cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)Tp, (cuuint64_t)H};
  cuuint64_t strides[2] = {(cuuint64_t)D * 2, (cuuint64_t)Tp * D * 2};
  cuuint32_t box[3] = {64, (cuuint32_t)box_rows, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = enc(m, fp16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, base, dims,
                   strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                   CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) { snprintf(err, errlen, "cuTensorMapEncodeTiled failed with CUresult %d", (int)r); return false; }
  return true;
}

}  // namespace

cudaError_t tc_prepare() {
  return cudaFuncSetAttribute(tc_attn_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SM_TOTAL);
}

TcMaps* tc_make_maps(const Geometry& g, const RotBuffers& rot, char* err, int errlen) {
  TcMaps* m = new TcMaps();
  bool ok = make_plane_map(&m->q_hi, rot.q_hi, g.Hq, g.Tp, BM, false, err, errlen) &&
            make_plane_map(&m->q_lo, rot.q_lo, g.Hq, g.Tp, BM, false, err, errlen) &&
            make_plane_map(&m->k_hi, rot.k_hi, g.Hkv, g.Tp, BN, false, err, errlen) &&
            make_plane_map(&m->k_lo, rot.k_lo, g.Hkv, g.Tp, BN, false, err, errlen) &&
            make_plane_map(&m->v, rot.v, g.Hkv, g.Tp, BN, true, err, errlen);
  if (!ok) { delete m; return nullptr; }
  return m;
}

void tc_free_maps(TcMaps* m) { delete m; }

cudaError_t tc_attention(const Geometry& g, const AttnArgs& a, const TcMaps* maps, cudaStream_t s) {
  if (a.n_items == 0) return cudaSuccess;
  dim3 grid(a.n_items, g.Hq);
  tc_attn_kernel<<<grid, THREADS, SM_TOTAL, s>>>(*maps, g, a);
  return cudaGetLastError();
}

}  // namespace lacache
