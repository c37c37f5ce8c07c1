// Token-wise producer in front of the first-layer attention (Sec. 3.3.2: embedding, attention norm,
// Q/K/V projections; the rotation of Eq. 1 is applied by the kernels that consume the result).
//
// Two kernels:
//   qkv_norm_kernel  one CTA per token: gathers the token's embedding row (or takes a given hidden
//                    state), RMS-normalises it in fp32 and writes the bf16 operand row X^ (and, on
//                    request, the embedding row itself: what the EmbedCache keeps).
//   qkv_gemm_kernel  Y^T = W X^T on tcgen05: the 128 output features of one head are the M rows of the
//                    MMA (A = a [128 x 64] tile of W, K-major, by TMA from a copy of W re-laid out at
//                    create so that every such tile is one contiguous 16 KB run), the tokens are its N columns
//                    (B = [TN x 64] tile of X^, K-major, by TMA), fp32 accumulators in TMEM.  With a
//                    block's 32..64 tokens the kernel is bound by reading W once from HBM, so the work
//                    is cut stream-K fashion: the (tile, 64-wide k chunk) pairs are dealt out in equal
//                    contiguous ranges to one persistent CTA per SM.  A CTA that owns only part of a
//                    tile's chunks leaves its fp32 partial in a workspace; the last CTA to arrive at a
//                    tile adds the partials in CTA order (the result does not depend on arrival order)
//                    and writes the bf16 rows.  With more CTAs than tiles and fewer than twice as many
//                    (a step at LLaDA width) the cut is by role instead, see GemmArgs::hp.  The kernel
//                    does not wait for the norm grid but for the count of operand rows it publishes,
//                    and for the grids ahead of it only before its final stores and its exit.
// Warp roles of the GEMM: warp 0 (one lane) TMA producer over a ring of stages, warp 1 (one lane) MMA
// issuer, warps 2..5 epilogue (TMEM lane = output feature).  Two accumulators alternate so that an
// epilogue overlaps the next segment's MMAs.  Every mbarrier wait is bounded; a wait that runs out sets
// the status word and the CTA unwinds (TMEM is always freed).
#include <cuda.h>
#include <cuda_bf16.h>
#include <stdarg.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <algorithm>
#include <new>

#include "lacache_internal.h"
#include "lacache_ptx.h"

using namespace lacache;

struct lacache_qkv {
  lacache_qkv_config cfg;
  int n_ftiles = 0;        // 128-row tiles of W = heads: Hq + 2 Hkv
  int tokens_pad = 0;      // rows of the operand buffer (max_tokens rounded up to 256)
  int num_sms = 148;
  int device = 0;
  __nv_bfloat16* w_packed = nullptr;    // W in tile order: [feature tile][k chunk][128 rows][64 columns]
  __nv_bfloat16* xhat = nullptr;        // [tokens_pad][d_model]
  float* ws = nullptr;                  // [3 * num_sms][256 * 128] partial tiles
  int* counters = nullptr;              // per tile: chunks accumulated so far
  int* ready = nullptr;                 // operand rows written so far, over all calls (wraps)
  unsigned ready_target = 0;            // what `ready` reads when the rows of the latest call are complete
  int32_t* status = nullptr;
  // scratch of the *_tokens calls, [max_tokens][H][128] each: the projections of all tokens (kept from
  // one build to the next, so that a build re-projects only the tokens that changed) and of a block
  __nv_bfloat16 *q = nullptr, *k = nullptr, *v = nullptr;
  __nv_bfloat16 *qb = nullptr, *kb = nullptr, *vb = nullptr;
  const void* full_owner = nullptr;     // the context whose tokens q / k / v currently hold
  int full_tokens = 0;
  CUtensorMap w_map;
  CUtensorMap x_map[4];                 // boxes of 32, 64, 128, 256 tokens
  cudaEvent_t ev_start = nullptr, ev_stop = nullptr;
  int last_launches = 0;
  // experiment knobs, read from the environment once at create
  long long wait_cycles = 0;  // limit of the projection kernel's waits (lacache_qkv_set_wait_limit); 0 = default
  bool no_pdl = false;        // LACACHE_NO_PDL: plain stream-ordered launches
  bool plain_split = false;   // LACACHE_QKV_PLAIN_SPLIT: no closer / helper roles
  char err[512];
};

namespace lacache {
namespace {

using namespace ptx;

constexpr int QD = 128;                 // head_dim = features per tile = MMA M
constexpr int BK = 64;                  // k chunk: one 128-byte swizzled row of bf16
constexpr int MAX_TN = 256;
constexpr int G_THREADS = 192;
constexpr int EPI_THREADS = 128;
constexpr uint32_t A_BYTES = QD * BK * 2;
constexpr int MAX_STAGES = 12;
constexpr int WS_SLOTS = 3;             // partial tiles a CTA may publish
constexpr uint32_t RING_BYTES = 229376;
constexpr uint32_t SMQ_BAR = RING_BYTES;
enum { QB_FULL = 0, QB_FREE = MAX_STAGES, QB_ACC_FULL = 2 * MAX_STAGES, QB_ACC_FREE = QB_ACC_FULL + 2,
       QB_N = QB_ACC_FREE + 2 };
constexpr uint32_t SMQ_TOTAL = SMQ_BAR + 8 * QB_N + 32;
static_assert(SMQ_TOTAL <= 232448, "exceeds the 227 KB per-CTA limit");
constexpr long long Q_WAIT_CYCLES = 4000000000ll;  // ~2 s: the default limit of every device-side wait
enum { QLOC_SMEM_ALIGN = 101, QLOC_WAIT_FULL = 102, QLOC_WAIT_FREE = 103, QLOC_WAIT_ACC_FULL = 104,
       QLOC_WAIT_ACC_FREE = 105, QLOC_TOKEN_ID = 106, QLOC_ROW = 107, QLOC_WAIT_ROWS = 108, QLOC_WAIT_PARTS = 109 };

struct GemmArgs {
  int n_tokens, tn, n_ttiles, n_tiles, kc;   // kc = d_model / 64 chunks per tile
  long long total_chunks;
  // Closer / helper split (hp > 0), used when there are more CTAs than tiles and fewer than twice as
  // many: n_tiles of the CTAs ("closers", the high block indices) own the last kc - hp chunks of one tile
  // each and finish it; the other CTAs ("helpers", placed first) share the first hp chunks of all tiles
  // in equal contiguous ranges and only publish partial tiles.  Helpers start earlier and get less work
  // than closers, so their parts are published by the time a closer is through: the closer fetches them
  // ahead of its last MMA and finishes its tile straight from TMEM, with no publish / count / read-back
  // round trips at the end of the kernel.
  int hp;
  int n_stages;
  int Hq, Hkv;
  __nv_bfloat16 *q, *k, *v;
  const int32_t* dst_rows;   // output row of input token t (null: t); rows outside [0, max_rows) are dropped
  int max_rows;
  const int* ready;          // count of operand rows the norm kernels have written (all calls, wraps)
  int ready_target;          // its value once this call's rows are complete
  float* ws;
  int* counters;
  int32_t* status;
  long long wait_cycles;     // limit of every device-side wait, in SM clock cycles
};

struct QCta {
  uint32_t base;
  volatile int* abort_flag;
  volatile int* rows_ready;   // set by the producer once the operand rows of this launch are complete
  int32_t* status;
  long long wait_cycles;      // limit of every wait of this launch
  __device__ __forceinline__ uint32_t bar(int slot) const { return base + SMQ_BAR + 8u * slot; }
};

__device__ __noinline__ bool q_wait_slow(const QCta& c, uint32_t bar, uint32_t parity, int loc) {
  long long t0 = clock64();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 32; ++i)
      if (mbar_try(bar, parity)) return true;
    if (*c.abort_flag) return false;
    if (clock64() - t0 > c.wait_cycles) {
      *c.abort_flag = 1;
      if (atomicCAS(c.status, 0, (int)LACACHE_ERR_TIMEOUT) == 0) {
        c.status[1] = loc;
        c.status[2] = blockIdx.x;
        c.status[3] = threadIdx.x;
      }
      return false;
    }
  }
}
__device__ __forceinline__ bool q_wait(const QCta& c, int slot, uint32_t parity, int loc) {
  const uint32_t b = c.bar(slot);
  if (mbar_try(b, parity)) return true;
  return q_wait_slow(c, b, parity, loc);
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1)
      : "memory");
}

// The CTAs that share a list of (tile, chunk) pairs in equal contiguous ranges: all CTAs and kc chunks per
// tile in the plain stream-K split; the helpers and the first hp chunks per tile in the closer / helper split.
struct Sharing {
  int n_ctas;        // CTAs that share the list
  int first_cta;     // block index of the first of them
  int kce;           // chunks per tile in the list
  long long total;   // n_tiles * kce
};
__device__ __forceinline__ Sharing sharing(const GemmArgs& a) {
  Sharing sh;
  if (a.hp > 0) { sh.n_ctas = (int)gridDim.x - a.n_tiles; sh.first_cta = 0; sh.kce = a.hp; }   // helpers are placed first
  else { sh.n_ctas = (int)gridDim.x; sh.first_cta = 0; sh.kce = a.kc; }
  sh.total = (long long)a.n_tiles * sh.kce;
  return sh;
}
// first list position of the j-th sharing CTA
__device__ __forceinline__ long long range_start(const Sharing& sh, int j) {
  return (long long)j * sh.total / (long long)sh.n_ctas;
}
// the sharing CTA (ordinal) whose range holds list position x
__device__ __forceinline__ int cta_of(const Sharing& sh, long long x) {
  return (int)(((x + 1) * (long long)sh.n_ctas - 1) / sh.total);
}
// This CTA's work: list positions [r0, r1) of a list with kce chunks per tile, whose chunk c is chunk
// coff + c of the tile.  A closer's list is its own: the last kc - hp chunks of every tile.
struct Work { long long r0, r1; int kce, coff; bool closer, helper; };
// BY_ROLE: the closer / helper split (a.hp > 0); a template parameter of the kernel, which then carries
// only the epilogue code of the split it runs
template <bool BY_ROLE>
__device__ __forceinline__ Work my_work(const GemmArgs& a) {
  Work w;
  const int b = (int)blockIdx.x;
  const int n_helpers = BY_ROLE ? (int)gridDim.x - a.n_tiles : 0;
  w.closer = BY_ROLE && b >= n_helpers;
  w.helper = BY_ROLE && b < n_helpers;
  if (w.closer) {
    w.kce = a.kc - a.hp; w.coff = a.hp;
    w.r0 = (long long)(b - n_helpers) * w.kce; w.r1 = w.r0 + w.kce;
  } else {
    const Sharing sh = sharing(a);
    w.kce = sh.kce; w.coff = 0;
    w.r0 = range_start(sh, b - sh.first_cta); w.r1 = range_start(sh, b - sh.first_cta + 1);
  }
  return w;
}

// destination of feature tile ft, input token t: a row of q, k or v (null: the row is dropped)
__device__ __forceinline__ __nv_bfloat16* out_row(const GemmArgs& a, int ft, int t) {
  if (a.dst_rows) {
    t = __ldg(a.dst_rows + t);
    if ((unsigned)t >= (unsigned)a.max_rows) return nullptr;   // reported by the norm kernel
  }
  if (ft < a.Hq) return a.q + ((size_t)t * a.Hq + ft) * QD;
  if (ft < a.Hq + a.Hkv) return a.k + ((size_t)t * a.Hkv + (ft - a.Hq)) * QD;
  return a.v + ((size_t)t * a.Hkv + (ft - a.Hq - a.Hkv)) * QD;
}

// Walks this CTA's chunks in order without divisions: ring stage and phase, tile coordinates, chunk.
struct ChunkCursor {
  int s; uint32_t ph;     // ring stage and its phase
  int ft, tt, ch;         // feature tile, token tile, k chunk
  int kce, coff;          // chunks per tile in this CTA's list; its chunk ch is chunk coff + ch of the tile
  __device__ __forceinline__ void init(const GemmArgs& a, const Work& w) {
    s = 0; ph = 0;
    kce = w.kce; coff = w.coff;
    const int tile = (int)(w.r0 / kce);
    ch = (int)(w.r0 % kce);
    ft = tile / a.n_ttiles;
    tt = tile % a.n_ttiles;
  }
  __device__ __forceinline__ void next(const GemmArgs& a) {
    if (++s == a.n_stages) { s = 0; ph ^= 1u; }
    if (++ch == kce) {
      ch = 0;
      if (++tt == a.n_ttiles) { tt = 0; ++ft; }
    }
  }
};

// Loads of one chunk into its ring stage: the W tile and / or the X^ tile.  One mbarrier per stage
// counts the bytes of both.
__device__ __forceinline__ void load_chunk(const QCta& c, const CUtensorMap* w_map, const CUtensorMap* x_map,
                                           const GemmArgs& a, const ChunkCursor& k, uint32_t stage_bytes,
                                           bool load_w, bool load_x) {
  const uint32_t dst = c.base + k.s * stage_bytes;
  if (load_w) {
    mbar_expect_tx(c.bar(QB_FULL + k.s), stage_bytes);
    tma_load_2d(dst, w_map, c.bar(QB_FULL + k.s), 0, (k.ft * a.kc + k.coff + k.ch) * QD);   // one contiguous 16 KB tile
  }
  if (load_x) tma_load_2d(dst + A_BYTES, x_map, c.bar(QB_FULL + k.s), (k.coff + k.ch) * BK, k.tt * a.tn);
}

// `early` chunks already have their W tile in flight (issued before the wait on the preceding grid)
__device__ __forceinline__ void gemm_producer(const QCta& c, const CUtensorMap* w_map, const CUtensorMap* x_map,
                                              const GemmArgs& a, const Work& w, uint32_t stage_bytes, int early) {
  // The operand rows X^ are written by the norm kernel launched just ahead, which counts the rows it has
  // completed.  Waiting for that count rather than for the whole grid lets this kernel work while grids
  // further ahead in the stream (a previous step's attention kernel, which the norm kernel may run
  // alongside) are still draining.  Every CTA of the norm kernel is resident by the time this kernel
  // starts (it lets its dependents launch at entry), so the count always arrives; the wait is bounded anyway.
  {
    const long long t_start = clock64();
    for (;;) {
      int cnt;
      asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(cnt) : "l"(a.ready) : "memory");
      if (cnt - a.ready_target >= 0) break;
      if (*c.abort_flag) return;
      if (clock64() - t_start > c.wait_cycles) {
        *c.abort_flag = 1;
        if (atomicCAS(c.status, 0, (int)LACACHE_ERR_TIMEOUT) == 0) {
          c.status[1] = QLOC_WAIT_ROWS; c.status[2] = blockIdx.x; c.status[3] = cnt;
        }
        return;
      }
    }
    asm volatile("fence.proxy.async.global;" ::: "memory");   // the rows are read through the async proxy (TMA)
    *c.rows_ready = 1;
  }
  ChunkCursor k;
  k.init(a, w);
  const int n = (int)(w.r1 - w.r0);
  for (int it = 0; it < n; ++it, k.next(a)) {
    if (it < early) {
      load_chunk(c, w_map, x_map, a, k, stage_bytes, false, true);
      continue;
    }
    if (!q_wait(c, QB_FREE + k.s, k.ph ^ 1u, QLOC_WAIT_FREE)) return;
    load_chunk(c, w_map, x_map, a, k, stage_bytes, true, true);
  }
}

__device__ __forceinline__ void gemm_mma(const QCta& c, const GemmArgs& a, uint32_t tmem, const Work& w,
                                         uint32_t stage_bytes) {
  const long long r0 = w.r0, r1 = w.r1;
  const uint32_t idesc = idesc_f16(1u /*bf16*/, 0u, QD, (uint32_t)a.tn);
  int s = 0;
  uint32_t ph = 0;
  int seg = 0;
  for (long long x = r0; x < r1; ++seg) {
    const int c0 = (int)(x % w.kce);
    const int c1 = (int)min((long long)w.kce, c0 + (r1 - x));
    const int buf = seg & 1;
    // the epilogue of the segment that used this accumulator two segments ago has drained it
    if (!q_wait(c, QB_ACC_FREE + buf, ((uint32_t)(seg >> 1) & 1u) ^ 1u, QLOC_WAIT_ACC_FREE)) return;
    tc_fence_after();
    const uint32_t acc = tmem + (uint32_t)(buf * MAX_TN);
    for (int ch = c0; ch < c1; ++ch) {
      if (!q_wait(c, QB_FULL + s, ph, QLOC_WAIT_FULL)) return;
      tc_fence_after();
      const uint32_t sa = c.base + s * stage_bytes;
      const uint64_t ad = smem_desc(sa, 16, 1024), bd = smem_desc(sa + A_BYTES, 16, 1024);
#pragma unroll
      for (int ks = 0; ks < BK / 16; ++ks)
        mma_ss(acc, ad + 2u * ks, bd + 2u * ks, idesc, (ch > c0 || ks > 0) ? 1u : 0u);
      tc_commit(c.bar(QB_FREE + s));
      if (++s == a.n_stages) { s = 0; ph ^= 1u; }
    }
    tc_commit(c.bar(QB_ACC_FULL + buf));
    x += c1 - c0;
  }
}

// A closer finishes its tile: the helpers' parts of the tile (published earlier, as a rule) are fetched
// ahead of the last MMA, then added to the accumulator straight from TMEM in ascending chunk order
// (helper parts first, then this CTA's chunks), rounded and stored.
__device__ __forceinline__ void closer_epilogue(const QCta& c, const GemmArgs& a, uint32_t tmem, const Work& w,
                                                volatile uint32_t* flag) {
  const int tid = threadIdx.x;
  const int et = tid - 64;
  const int quad = (tid >> 5) & 3;
  const int f = quad * 32 + (tid & 31);
  const uint32_t lane_off = (uint32_t)(quad * 32) << 16;
  const int tile = (int)blockIdx.x - ((int)gridDim.x - a.n_tiles);
  const int ft = tile / a.n_ttiles, tt = tile % a.n_ttiles;
  const int t0 = tt * a.tn;
  const int nt = min(a.tn, a.n_tokens - t0);
  // Every helper part of the tile has been published once the tile's counter shows all hp chunks.  The
  // counter is looked at only after this launch's operand rows are complete: every earlier launch of the
  // handle (whose closer may not have reset the counter yet) is then over.
  if (et == 0) {
    const long long t_start = clock64();
    uint32_t ok = 1;
    for (;;) {
      int cnt = -1;
      if (*c.rows_ready)
        asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(cnt) : "l"(a.counters + tile) : "memory");
      if (cnt == a.hp) break;
      if (*c.abort_flag) { ok = 0; break; }
      if (clock64() - t_start > c.wait_cycles) {
        *c.abort_flag = 1;
        if (atomicCAS(c.status, 0, (int)LACACHE_ERR_TIMEOUT) == 0) {
          c.status[1] = QLOC_WAIT_PARTS; c.status[2] = blockIdx.x; c.status[3] = cnt;
        }
        ok = 0;
        break;
      }
    }
    if (ok) a.counters[tile] = 0;                  // ready for the next launch
    *flag = ok;
  }
  asm volatile("bar.sync 1, 128;" ::: "memory");
  if (*flag == 0) return;
  __threadfence();
  // the helpers whose ranges touch the first hp chunks of this tile, in ascending order (at most three:
  // a helper's range is at least hp long)
  const Sharing sh = sharing(a);
  const long long x_lo = (long long)tile * sh.kce;
  const int j_lo = cta_of(sh, x_lo), j_hi = cta_of(sh, x_lo + sh.kce - 1);
  const float *p0 = nullptr, *p1 = nullptr, *p2 = nullptr;
  int n_parts = 0;
  for (int j = j_lo; j <= j_hi; ++j) {
    const long long s0 = range_start(sh, j), s1 = range_start(sh, j + 1);
    if (s1 <= s0) continue;
    const int slot = tile - (int)(s0 / sh.kce);    // the ordinal of this tile among the helper's segments
    const float* p = a.ws + ((size_t)(sh.first_cta + j) * WS_SLOTS + slot) * (size_t)(MAX_TN * QD) + f;
    if (n_parts == 0) p0 = p; else if (n_parts == 1) p1 = p; else p2 = p;
    ++n_parts;
  }
  for (int g = 0; g * 32 < nt; ++g) {
    float pre0[32], pre1[32], pre2[32];
#pragma unroll
    for (int i = 0; i < 32; ++i) {
      const int t = g * 32 + i;
      const size_t o = (size_t)t * QD;
      pre0[i] = (t < nt && n_parts > 0) ? __ldcg(p0 + o) : 0.f;
      pre1[i] = (t < nt && n_parts > 1) ? __ldcg(p1 + o) : 0.f;
      pre2[i] = (t < nt && n_parts > 2) ? __ldcg(p2 + o) : 0.f;
    }
    if (g == 0) {
      if (!q_wait(c, QB_ACC_FULL, 0, QLOC_WAIT_ACC_FULL)) return;
      tc_fence_after();
      grid_dependency_wait();   // results may overwrite rows that a grid ahead in the stream still reads
    }
    uint32_t r[32];
    tmem_ld32(tmem + lane_off + (uint32_t)(g * 32), r);
    tmem_ld_wait();
#pragma unroll
    for (int i = 0; i < 32; ++i) {
      const int t = g * 32 + i;
      float sum = 0.f + pre0[i];
      if (n_parts > 1) sum += pre1[i];
      if (n_parts > 2) sum += pre2[i];
      sum += __uint_as_float(r[i]);
      if (t < nt) {
        __nv_bfloat16* dst = out_row(a, ft, t0 + t);
        if (dst) dst[f] = __float2bfloat16_rn(sum);
      }
    }
  }
  tc_fence_before();
  mbar_arrive(c.bar(QB_ACC_FREE));
}

template <bool BY_ROLE>
__device__ __forceinline__ void gemm_epilogue(const QCta& c, const GemmArgs& a, uint32_t tmem, const Work& w,
                                              volatile uint32_t* flag) {
  if (BY_ROLE && w.closer) { closer_epilogue(c, a, tmem, w, flag); return; }
  const long long r0 = w.r0, r1 = w.r1;
  const Sharing sh = sharing(a);
  const int tid = threadIdx.x;
  const int et = tid - 64;                       // 0..127
  const int quad = (tid >> 5) & 3;               // the TMEM lane quadrant this warp may read
  const int f = quad * 32 + (tid & 31);          // output feature within the tile
  const uint32_t lane_off = (uint32_t)(quad * 32) << 16;
  int seg = 0;
  for (long long x = r0; x < r1; ++seg) {
    const int tile = (int)(x / w.kce), c0 = (int)(x % w.kce);
    const int c1 = (int)min((long long)w.kce, c0 + (r1 - x));
    const int ft = tile / a.n_ttiles, tt = tile % a.n_ttiles;
    const int t0 = tt * a.tn;
    const int nt = min(a.tn, a.n_tokens - t0);   // valid tokens of the tile
    const int buf = seg & 1;
    const bool whole = !BY_ROLE && (c0 == 0 && c1 == a.kc);
    if (!q_wait(c, QB_ACC_FULL + buf, (uint32_t)(seg >> 1) & 1u, QLOC_WAIT_ACC_FULL)) return;
    tc_fence_after();
    // plain split: a CTA's range leaves at most its first and its last segment partial (slots 0 and 1);
    // a helper publishes every segment, of which it has at most three
    float* part = a.ws + ((size_t)blockIdx.x * WS_SLOTS + (BY_ROLE ? seg : (seg == 0 ? 0 : 1))) * (size_t)(MAX_TN * QD);
    for (int g = 0; g * 32 < nt; ++g) {
      uint32_t r[32];
      tmem_ld32(tmem + lane_off + (uint32_t)(buf * MAX_TN + g * 32), r);
      tmem_ld_wait();
      if (whole) {
        grid_dependency_wait();   // results may overwrite rows that a grid ahead in the stream still reads
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          const int t = g * 32 + i;
          if (t < nt) {
            __nv_bfloat16* dst = out_row(a, ft, t0 + t);
            if (dst) dst[f] = __float2bfloat16_rn(__uint_as_float(r[i]));
          }
        }
      } else {
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          const int t = g * 32 + i;
          if (t < nt) part[(size_t)t * QD + f] = __uint_as_float(r[i]);
        }
      }
    }
    tc_fence_before();
    mbar_arrive(c.bar(QB_ACC_FREE + buf));
    if (!whole) {
      // publish the partial, then count this segment's chunks; whoever completes the tile adds up
      __threadfence();
      asm volatile("bar.sync 1, 128;" ::: "memory");
      if (et == 0) {
        const int old = atomicAdd(a.counters + tile, c1 - c0);
        // (a helper's tiles are finished by their closers)
        const uint32_t last = (!BY_ROLE && old + (c1 - c0) == a.kc) ? 1u : 0u;
        if (last) a.counters[tile] = 0;           // ready for the next launch
        *flag = last;
      }
      asm volatile("bar.sync 1, 128;" ::: "memory");
      if (*flag) {
        grid_dependency_wait();   // results may overwrite rows that a grid ahead in the stream still reads
        __threadfence();
        // four features per thread, four token rows per pass of the 128 threads; the loads of eight
        // passes (32 tokens) are issued together so that the tile costs a few memory round trips
        const long long x_lo = (long long)tile * a.kc, x_hi = x_lo + a.kc;
        const int j_lo = cta_of(sh, x_lo), j_hi = cta_of(sh, x_hi - 1);
        const int f4 = (et & 31) * 4, tr = et >> 5;
        // the tile's parts in ascending CTA order (a fixed summation order); with up to three of them,
        // the usual case, the loads of all parts are in flight together
        const float *p0 = nullptr, *p1 = nullptr, *p2 = nullptr;
        int n_parts = 0;
        for (int j = j_lo; j <= j_hi; ++j) {
          const long long s0 = range_start(sh, j), s1 = range_start(sh, j + 1);
          if (s1 <= s0) continue;                   // a CTA without work
          const int slot = (s0 >= x_lo) ? 0 : 1;    // the tile holds its first segment, or its last
          const float* p = a.ws + ((size_t)j * WS_SLOTS + slot) * (size_t)(MAX_TN * QD) + f4;
          if (n_parts == 0) p0 = p; else if (n_parts == 1) p1 = p; else if (n_parts == 2) p2 = p;
          ++n_parts;
        }
        const float4 zero4 = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int tb = 0; tb < nt; tb += 32) {
          float4 acc[8];
          if (n_parts <= 3) {
            float4 v0[8], v1[8], v2[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              const int t = tb + tr + 4 * i;
              const size_t o = (size_t)t * QD;
              v0[i] = (t < nt) ? __ldcg(reinterpret_cast<const float4*>(p0 + o)) : zero4;
              v1[i] = (t < nt && n_parts > 1) ? __ldcg(reinterpret_cast<const float4*>(p1 + o)) : zero4;
              v2[i] = (t < nt && n_parts > 2) ? __ldcg(reinterpret_cast<const float4*>(p2 + o)) : zero4;
            }
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              acc[i].x = 0.f + v0[i].x; acc[i].y = 0.f + v0[i].y; acc[i].z = 0.f + v0[i].z; acc[i].w = 0.f + v0[i].w;
              if (n_parts > 1) { acc[i].x += v1[i].x; acc[i].y += v1[i].y; acc[i].z += v1[i].z; acc[i].w += v1[i].w; }
              if (n_parts > 2) { acc[i].x += v2[i].x; acc[i].y += v2[i].y; acc[i].z += v2[i].z; acc[i].w += v2[i].w; }
            }
          } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) acc[i] = zero4;
            for (int j = j_lo; j <= j_hi; ++j) {
              const long long s0 = range_start(sh, j), s1 = range_start(sh, j + 1);
              if (s1 <= s0) continue;
              const int slot = (s0 >= x_lo) ? 0 : 1;
              const float* p = a.ws + ((size_t)j * WS_SLOTS + slot) * (size_t)(MAX_TN * QD) + f4;
              float4 v[8];
#pragma unroll
              for (int i = 0; i < 8; ++i) {
                const int t = tb + tr + 4 * i;
                v[i] = (t < nt) ? __ldcg(reinterpret_cast<const float4*>(p + (size_t)t * QD)) : zero4;
              }
#pragma unroll
              for (int i = 0; i < 8; ++i) {
                acc[i].x += v[i].x; acc[i].y += v[i].y; acc[i].z += v[i].z; acc[i].w += v[i].w;
              }
            }
          }
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const int t = tb + tr + 4 * i;
            if (t < nt) {
              __nv_bfloat162 lo = __floats2bfloat162_rn(acc[i].x, acc[i].y), hi = __floats2bfloat162_rn(acc[i].z, acc[i].w);
              uint2 o;
              o.x = *reinterpret_cast<uint32_t*>(&lo);
              o.y = *reinterpret_cast<uint32_t*>(&hi);
              __nv_bfloat16* dst = out_row(a, ft, t0 + t);
              if (dst) *reinterpret_cast<uint2*>(dst + f4) = o;
            }
          }
        }
      }
      asm volatile("bar.sync 1, 128;" ::: "memory");   // the flag word is reused by the next segment
    }
    x += c1 - c0;
  }
}

template <bool BY_ROLE>
__global__ void __launch_bounds__(G_THREADS, 1)
qkv_gemm_kernel(const __grid_constant__ CUtensorMap w_map, const __grid_constant__ CUtensorMap x_map,
                const GemmArgs a) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const int tid = threadIdx.x;
  const int warp = tid >> 5;
  // a kernel launched programmatically dependent on this one may be scheduled now (it has to wait
  // for this grid before it touches anything this grid writes)
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  QCta c;
  c.base = smem_u32(smem_raw);
  uint32_t* words = reinterpret_cast<uint32_t*>(smem_raw + SMQ_BAR + 8 * QB_N);  // [0] tmem, [1] abort, [2] flag
  c.abort_flag = reinterpret_cast<volatile int*>(words + 1);
  c.rows_ready = reinterpret_cast<volatile int*>(words + 3);
  c.status = a.status;
  c.wait_cycles = a.wait_cycles;
  if ((c.base & 1023u) != 0) {
    if (tid == 0 && atomicCAS(a.status, 0, (int)LACACHE_ERR_CUDA) == 0) a.status[1] = QLOC_SMEM_ALIGN;
    return;
  }
  const Work w = my_work<BY_ROLE>(a);
  const long long r0 = w.r0, r1 = w.r1;
  const uint32_t stage_bytes = A_BYTES + (uint32_t)a.tn * 128u;
  int early = 0;
  if (tid == 0) {
    prefetch_map(&w_map);
    prefetch_map(&x_map);
    for (int i = 0; i < QB_N; ++i) mbar_init(c.bar(i), (i >= QB_ACC_FREE) ? EPI_THREADS : 1);
    words[1] = 0;
    words[2] = 0;
    words[3] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_async_smem();
    // the weights do not depend on the kernel before this one: fill the ring with W tiles right away
    // (the X^ tiles of the same stages follow after the wait below)
    early = (int)min((long long)a.n_stages, r1 - r0);
    ChunkCursor k;
    k.init(a, w);
    for (int it = 0; it < early; ++it, k.next(a)) load_chunk(c, &w_map, &x_map, a, k, stage_bytes, true, false);
  }
  __syncwarp();
  if (warp == 1) {  // (warp 1 allocates while thread 0 is still initialising barriers and requesting weights)
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(words)), "r"(512)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = words[0];

  if (warp == 0) {
    if (tid == 0) gemm_producer(c, &w_map, &x_map, a, w, stage_bytes, early);
  } else if (warp == 1) {
    if (tid == 32) gemm_mma(c, a, tmem, w, stage_bytes);
  } else {
    gemm_epilogue<BY_ROLE>(c, a, tmem, w, words + 2);
  }
  __syncwarp();
  // this grid must not complete before the grids ahead of it have: whatever waits for it relies on that
  grid_dependency_wait();
  // teardown: free TMEM once every thread is past its last TMEM access
  if (*c.abort_flag) {
    // a bounded wait ran out: copies requested before that may still be on their way into this CTA's shared
    // memory; give them time to land (a fixed 50 us) before it is given up
    const long long t0 = clock64();
    while (clock64() - t0 < 100000ll) {
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {  // the warp that allocated
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512) : "memory");
  }
}

// W [rows][d_model] -> tile order [rows / 128][d_model / 64][128][64]: every (feature tile, k chunk)
// operand tile becomes one contiguous 16 KB run, so that the projection streams W from HBM in
// whole DRAM pages instead of 128-byte pieces a row pitch apart.  Runs once, at create.
__global__ void qkv_pack_w_kernel(const uint4* __restrict__ w, uint4* __restrict__ wp, int rows, int d_model) {
  const int per_row = d_model / 8;                       // 16-byte pieces per row
  const size_t n = (size_t)rows * per_row;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
    const int r = (int)(i / per_row), p = (int)(i % per_row);
    const int ft = r / QD, rr = r % QD, ch = p / 8, pp = p % 8;
    wp[(((size_t)ft * (d_model / BK) + ch) * QD + rr) * 8 + pp] = w[i];
  }
}

// ---------------------------------------------------------------------------------------------------
constexpr int N_THREADS = 256;
constexpr int N_MAX_CHUNKS = 4;   // 8-element chunks per thread: d_model <= 8192

struct NormArgs {
  const int32_t* ids;             // or null
  const __nv_bfloat16* hidden;    // [n][d_model], used when ids == null
  const __nv_bfloat16* table;     // [vocab][d_model]
  const __nv_bfloat16* weight;    // [d_model]
  __nv_bfloat16* xhat;            // [n][d_model]
  __nv_bfloat16* h_out;           // [n][d_model] or null
  const int32_t* dst_rows;        // or null; checked against max_rows here
  int max_rows;
  int* ready;                     // incremented once this row of X^ is complete and visible
  int early_inputs;               // the inputs were complete before the preceding grid started: read them at once
  int d_model, vocab;
  float eps;
  int32_t* status;
};

__global__ void __launch_bounds__(N_THREADS) qkv_norm_kernel(const NormArgs a) {
  // The projection kernel may be scheduled now: before it waits for this grid it only sets itself up
  // and starts fetching weights.  This kernel is itself launched programmatically dependent and waits,
  // before its first load, for everything enqueued ahead of it (whatever wrote the token ids or hidden
  // states included); the projection kernel's own wait then covers all of that as well.
  // (A caller that vouches for inputs that were complete before the grid ahead was even enqueued gets
  // the wait at the end instead: this kernel then runs alongside that grid, and still does not complete
  // before it, which is what the projection kernel's wait relies on.  The operand rows X^ it writes are
  // read by nothing but the projection kernel of this call.)
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (!a.early_inputs) grid_dependency_wait();
  __shared__ float red[N_THREADS / 32];
  const int t = blockIdx.x;
  const int tid = threadIdx.x;
  const __nv_bfloat16* src;
  bool valid = true;
  if (a.dst_rows && tid == 0) {
    const int row = a.dst_rows[t];
    if ((unsigned)row >= (unsigned)a.max_rows && atomicCAS(a.status, 0, (int)LACACHE_ERR_INVALID_ARG) == 0) {
      a.status[1] = QLOC_ROW;
      a.status[2] = t;
      a.status[3] = row;
    }
  }
  if (a.ids) {
    const int id = a.ids[t];
    valid = id >= 0 && id < a.vocab;
    if (!valid && tid == 0 && atomicCAS(a.status, 0, (int)LACACHE_ERR_INVALID_ARG) == 0) {
      a.status[1] = QLOC_TOKEN_ID;
      a.status[2] = t;
      a.status[3] = id;
    }
    src = a.table + (size_t)(valid ? id : 0) * a.d_model;
  } else {
    src = a.hidden + (size_t)t * a.d_model;
  }
  const int n_chunks = a.d_model / 8;
  uint4 raw[N_MAX_CHUNKS];
  float ss = 0.f;
#pragma unroll
  for (int i = 0; i < N_MAX_CHUNKS; ++i) {
    const int ch = tid + i * N_THREADS;
    raw[i] = make_uint4(0, 0, 0, 0);
    if (ch < n_chunks && valid) raw[i] = __ldg(reinterpret_cast<const uint4*>(src) + ch);
    const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(&raw[i]);
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const float2 x = __bfloat1622float2(p[e]);
      ss = fmaf(x.x, x.x, ss);
      ss = fmaf(x.y, x.y, ss);
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
  if ((tid & 31) == 0) red[tid >> 5] = ss;
  __syncthreads();
  float tot = 0.f;
#pragma unroll
  for (int i = 0; i < N_THREADS / 32; ++i) tot += red[i];
  // an invalid token id (reported through the status word) yields a zero row
  const float rinv = valid ? 1.0f / sqrtf(tot / (float)a.d_model + a.eps) : 0.f;
#pragma unroll
  for (int i = 0; i < N_MAX_CHUNKS; ++i) {
    const int ch = tid + i * N_THREADS;
    if (ch >= n_chunks) continue;
    const uint4 wraw = __ldg(reinterpret_cast<const uint4*>(a.weight) + ch);
    const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(&raw[i]);
    const __nv_bfloat162* w = reinterpret_cast<const __nv_bfloat162*>(&wraw);
    uint4 o;
    __nv_bfloat162* q = reinterpret_cast<__nv_bfloat162*>(&o);
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const float2 x = __bfloat1622float2(p[e]);
      const float2 g = __bfloat1622float2(w[e]);
      q[e] = __floats2bfloat162_rn(x.x * rinv * g.x, x.y * rinv * g.y);
    }
    reinterpret_cast<uint4*>(a.xhat + (size_t)t * a.d_model)[ch] = o;
    if (a.h_out && !a.early_inputs) reinterpret_cast<uint4*>(a.h_out + (size_t)t * a.d_model)[ch] = raw[i];
  }
  // publish the row: every thread's stores, then one count
  __threadfence();
  __syncthreads();
  if (tid == 0) atomicAdd(a.ready, 1);
  if (a.early_inputs) {
    grid_dependency_wait();
    if (a.h_out) {   // a caller's buffer: not before the grids ahead are complete
#pragma unroll
      for (int i = 0; i < N_MAX_CHUNKS; ++i) {
        const int ch = tid + i * N_THREADS;
        if (ch < n_chunks) reinterpret_cast<uint4*>(a.h_out + (size_t)t * a.d_model)[ch] = raw[i];
      }
    }
  }
}

// ---------------------------------------------------------------------------------------------------
thread_local char g_qkv_create_err[512] = "";

lacache_status qfail(lacache_qkv* p, lacache_status st, const char* fmt, ...) {
  char* dst = p ? p->err : g_qkv_create_err;
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(dst, 512, fmt, ap);
  va_end(ap);
  return st;
}

#define QCU_TRY(p, expr)                                                               \
  do {                                                                                 \
    cudaError_t e_ = (expr);                                                           \
    if (e_ != cudaSuccess)                                                             \
      return qfail(p, e_ == cudaErrorMemoryAllocation ? LACACHE_ERR_OOM : LACACHE_ERR_CUDA, \
                   "%s: %s", #expr, cudaGetErrorString(e_));                           \
  } while (0)

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// bf16 matrix [rows][cols] row-major as a 2-D tensor {cols, rows}; box = 64 columns x box_rows rows
bool make_bf16_map(lacache_qkv* p, CUtensorMap* m, const void* base, int rows, int cols, int box_rows) {
  static EncodeTiledFn enc = nullptr;
  if (!enc) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess) {
      qfail(p, LACACHE_ERR_CUDA, "cuTensorMapEncodeTiled entry point not found");
      return false;
    }
    enc = reinterpret_cast<EncodeTiledFn>(fn);
  }
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
  cuuint32_t box[2] = {(cuuint32_t)BK, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    qfail(p, LACACHE_ERR_CUDA, "cuTensorMapEncodeTiled (2-D bf16) failed with CUresult %d", (int)r);
    return false;
  }
  return true;
}

void qkv_free(lacache_qkv* p) {
  if (!p) return;
  cudaDeviceSynchronize();
  void* bufs[] = {p->w_packed, p->xhat, p->ws, p->counters, p->ready, p->status, p->q, p->k, p->v, p->qb, p->kb, p->vb};
  for (void* b : bufs)
    if (b) cudaFree(b);
  delete p;
}

bool misaligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; }

}  // namespace

// scratch rows the *_tokens entry points project into: all tokens of a context, or a block
void qkv_scratch(lacache_qkv* p, bool block, void** q, void** k, void** v) {
  *q = block ? p->qb : p->q; *k = block ? p->kb : p->k; *v = block ? p->vb : p->v;
}
void qkv_set_full_owner(lacache_qkv* p, const void* ctx, int n_tokens) { p->full_owner = ctx; p->full_tokens = n_tokens; }
bool qkv_full_owner_is(const lacache_qkv* p, const void* ctx, int n_tokens) {
  return p->full_owner == ctx && p->full_tokens == n_tokens;
}
int qkv_heads(const lacache_qkv* p, int* hq, int* hkv, int* max_tokens) {
  *hq = p->cfg.n_q_heads; *hkv = p->cfg.n_kv_heads; *max_tokens = p->cfg.max_tokens;
  return p->cfg.head_dim;
}

}  // namespace lacache

extern "C" {

lacache_status lacache_qkv_create(const lacache_qkv_config* cfg, lacache_qkv** out) {
  if (out) *out = nullptr;
  if (!cfg || !out) return qfail(nullptr, LACACHE_ERR_INVALID_ARG, "NULL argument");
  if (cfg->head_dim != QD) return qfail(nullptr, LACACHE_ERR_UNSUPPORTED, "head_dim %d: only 128", cfg->head_dim);
  if (cfg->d_model < BK || cfg->d_model % BK != 0 || cfg->d_model > 8 * N_THREADS * N_MAX_CHUNKS)
    return qfail(nullptr, LACACHE_ERR_SHAPE, "d_model %d: a multiple of 64 in [64, 8192]", cfg->d_model);
  if (cfg->n_q_heads < 1 || cfg->n_kv_heads < 1 || cfg->n_q_heads % cfg->n_kv_heads != 0)
    return qfail(nullptr, LACACHE_ERR_SHAPE, "heads %d / %d", cfg->n_q_heads, cfg->n_kv_heads);
  if (cfg->max_tokens < 1 || cfg->vocab < 0 || !(cfg->rms_eps >= 0.f))
    return qfail(nullptr, LACACHE_ERR_INVALID_ARG, "max_tokens %d, vocab %d, rms_eps %g", cfg->max_tokens, cfg->vocab,
                 (double)cfg->rms_eps);
  if (!cfg->norm_weight || !cfg->w_qkv || (cfg->vocab > 0 && !cfg->embed))
    return qfail(nullptr, LACACHE_ERR_INVALID_ARG, "NULL weight pointer");
  if (misaligned16(cfg->norm_weight) || misaligned16(cfg->w_qkv) || misaligned16(cfg->embed))
    return qfail(nullptr, LACACHE_ERR_INVALID_ARG, "weight pointer not 16-byte aligned");
  int n_dev = 0;
  if (cudaGetDeviceCount(&n_dev) != cudaSuccess || n_dev < 1) {
    cudaGetLastError();
    return qfail(nullptr, LACACHE_ERR_CUDA, "no CUDA device");
  }
  lacache_qkv* p = new (std::nothrow) lacache_qkv();
  if (!p) return qfail(nullptr, LACACHE_ERR_OOM, "host allocation failed");
  p->cfg = *cfg;
  p->err[0] = 0;
  p->n_ftiles = cfg->n_q_heads + 2 * cfg->n_kv_heads;
  p->tokens_pad = (cfg->max_tokens + MAX_TN - 1) / MAX_TN * MAX_TN;
  lacache_status st = LACACHE_OK;
  auto attempt = [&]() -> lacache_status {
    p->no_pdl = getenv("LACACHE_NO_PDL") != nullptr;
    p->plain_split = getenv("LACACHE_QKV_PLAIN_SPLIT") != nullptr;
    QCU_TRY(p, cudaGetDevice(&p->device));
    cudaDeviceProp prop;
    QCU_TRY(p, cudaGetDeviceProperties(&prop, p->device));
    if (prop.major != 10) return qfail(p, LACACHE_ERR_UNSUPPORTED, "device is sm_%d%d, need sm_100", prop.major, prop.minor);
    p->num_sms = prop.multiProcessorCount;
    const size_t d = (size_t)cfg->d_model;
    QCU_TRY(p, cudaMalloc(&p->xhat, (size_t)p->tokens_pad * d * 2));
    QCU_TRY(p, cudaMemset(p->xhat, 0, (size_t)p->tokens_pad * d * 2));
    QCU_TRY(p, cudaMalloc(&p->ws, (size_t)WS_SLOTS * p->num_sms * MAX_TN * QD * 4));
    const int max_tiles = p->n_ftiles * ((cfg->max_tokens + 31) / 32);
    QCU_TRY(p, cudaMalloc(&p->counters, (size_t)max_tiles * 4));
    QCU_TRY(p, cudaMemset(p->counters, 0, (size_t)max_tiles * 4));
    QCU_TRY(p, cudaMalloc(&p->ready, 4));
    QCU_TRY(p, cudaMemset(p->ready, 0, 4));
    QCU_TRY(p, cudaMalloc(&p->status, 16));
    QCU_TRY(p, cudaMemset(p->status, 0, 16));
    QCU_TRY(p, cudaMalloc(&p->q, (size_t)cfg->max_tokens * cfg->n_q_heads * QD * 2));
    QCU_TRY(p, cudaMalloc(&p->k, (size_t)cfg->max_tokens * cfg->n_kv_heads * QD * 2));
    QCU_TRY(p, cudaMalloc(&p->v, (size_t)cfg->max_tokens * cfg->n_kv_heads * QD * 2));
    QCU_TRY(p, cudaMalloc(&p->qb, (size_t)cfg->max_tokens * cfg->n_q_heads * QD * 2));
    QCU_TRY(p, cudaMalloc(&p->kb, (size_t)cfg->max_tokens * cfg->n_kv_heads * QD * 2));
    QCU_TRY(p, cudaMalloc(&p->vb, (size_t)cfg->max_tokens * cfg->n_kv_heads * QD * 2));
    const int w_rows = p->n_ftiles * QD;
    QCU_TRY(p, cudaMalloc(&p->w_packed, (size_t)w_rows * d * 2));
    qkv_pack_w_kernel<<<p->num_sms * 8, 256>>>(reinterpret_cast<const uint4*>(cfg->w_qkv),
                                               reinterpret_cast<uint4*>(p->w_packed), w_rows, cfg->d_model);
    QCU_TRY(p, cudaGetLastError());
    QCU_TRY(p, cudaDeviceSynchronize());
    // the packed copy as a matrix of 64 columns: a tile is 128 consecutive rows
    if (!make_bf16_map(p, &p->w_map, p->w_packed, w_rows * (cfg->d_model / BK), BK, QD)) return LACACHE_ERR_CUDA;
    for (int i = 0; i < 4; ++i)
      if (!make_bf16_map(p, &p->x_map[i], p->xhat, p->tokens_pad, cfg->d_model, 32 << i)) return LACACHE_ERR_CUDA;
    QCU_TRY(p, cudaFuncSetAttribute(qkv_gemm_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMQ_TOTAL));
    QCU_TRY(p, cudaFuncSetAttribute(qkv_gemm_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMQ_TOTAL));
    return LACACHE_OK;
  };
  st = attempt();
  if (st != LACACHE_OK) {
    snprintf(g_qkv_create_err, sizeof g_qkv_create_err, "%s", p->err);
    qkv_free(p);
    return st;
  }
  *out = p;
  return LACACHE_OK;
}

lacache_status lacache_qkv_destroy(lacache_qkv* p) {
  if (!p) return LACACHE_ERR_INVALID_ARG;
  qkv_free(p);
  return LACACHE_OK;
}

lacache_status lacache_qkv_project(lacache_qkv* p, const int32_t* token_ids, const void* hidden, int n_tokens,
                                   void* q, void* k, void* v, void* h_out, void* stream) {
  return lacache::qkv_project_rows(p, token_ids, hidden, n_tokens, q, k, v, h_out, nullptr, 0, false, stream);
}

}  // extern "C"

namespace lacache {
namespace {
lacache_status project_impl(lacache_qkv* p, const int32_t* token_ids, const void* hidden, int n_tokens, void* q,
                            void* k, void* v, void* h_out, const int32_t* dst_rows, int max_rows, bool early_inputs,
                            void* stream, bool without_norm);
}
lacache_status qkv_project_rows(lacache_qkv* p, const int32_t* token_ids, const void* hidden, int n_tokens, void* q,
                                void* k, void* v, void* h_out, const int32_t* dst_rows, int max_rows, bool early_inputs,
                                void* stream) {
  return project_impl(p, token_ids, hidden, n_tokens, q, k, v, h_out, dst_rows, max_rows, early_inputs, stream, false);
}
namespace {
lacache_status project_impl(lacache_qkv* p, const int32_t* token_ids, const void* hidden, int n_tokens, void* q,
                            void* k, void* v, void* h_out, const int32_t* dst_rows, int max_rows, bool early_inputs,
                            void* stream, bool without_norm) {
  if (!p) return LACACHE_ERR_INVALID_ARG;
  if ((token_ids == nullptr) == (hidden == nullptr))
    return qfail(p, LACACHE_ERR_INVALID_ARG, "pass exactly one of token_ids and hidden");
  if (token_ids && p->cfg.vocab == 0) return qfail(p, LACACHE_ERR_STATE, "token ids given but no embedding table");
  if (!q || !k || !v) return qfail(p, LACACHE_ERR_INVALID_ARG, "NULL output pointer");
  if (misaligned16(q) || misaligned16(k) || misaligned16(v) || misaligned16(hidden) || misaligned16(h_out))
    return qfail(p, LACACHE_ERR_INVALID_ARG, "pointer not 16-byte aligned");
  if (n_tokens < 0 || n_tokens > p->cfg.max_tokens)
    return qfail(p, LACACHE_ERR_SHAPE, "n_tokens %d outside [0, %d]", n_tokens, p->cfg.max_tokens);
  p->last_launches = 0;
  if (n_tokens == 0) return LACACHE_OK;
  cudaStream_t s = (cudaStream_t)stream;

  NormArgs na{};
  na.ids = token_ids;
  na.hidden = reinterpret_cast<const __nv_bfloat16*>(hidden);
  na.table = reinterpret_cast<const __nv_bfloat16*>(p->cfg.embed);
  na.weight = reinterpret_cast<const __nv_bfloat16*>(p->cfg.norm_weight);
  na.xhat = p->xhat;
  na.h_out = reinterpret_cast<__nv_bfloat16*>(h_out);
  na.dst_rows = dst_rows;
  na.max_rows = max_rows;
  na.early_inputs = early_inputs ? 1 : 0;
  na.ready = p->ready;
  na.d_model = p->cfg.d_model;
  na.vocab = p->cfg.vocab;
  na.eps = p->cfg.rms_eps;
  na.status = p->status;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  const bool no_pdl = p->no_pdl;
  if (!without_norm) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(n_tokens);
    cfg.blockDim = dim3(N_THREADS);
    cfg.stream = s;
    cfg.attrs = attr;
    cfg.numAttrs = no_pdl ? 0 : 1;
    QCU_TRY(p, cudaLaunchKernelEx(&cfg, qkv_norm_kernel, na));
  }
  // the norm kernel is enqueued and will publish its n_tokens rows: only now does the count the
  // projection waits for move (a failed launch above leaves counter and target in step)
  if (!without_norm) {
    p->ready_target += (unsigned)n_tokens;
    p->last_launches++;
  }

  GemmArgs ga{};
  int tn_idx = 0;
  while (tn_idx < 3 && (32 << tn_idx) < n_tokens) ++tn_idx;
  ga.n_tokens = n_tokens;
  ga.tn = 32 << tn_idx;
  ga.n_ttiles = (n_tokens + ga.tn - 1) / ga.tn;
  ga.n_tiles = p->n_ftiles * ga.n_ttiles;
  ga.kc = p->cfg.d_model / BK;
  ga.total_chunks = (long long)ga.n_tiles * ga.kc;
  ga.n_stages = (int)std::min<uint32_t>(MAX_STAGES, RING_BYTES / (A_BYTES + (uint32_t)ga.tn * 128u));
  ga.Hq = p->cfg.n_q_heads;
  ga.Hkv = p->cfg.n_kv_heads;
  ga.q = reinterpret_cast<__nv_bfloat16*>(q);
  ga.k = reinterpret_cast<__nv_bfloat16*>(k);
  ga.v = reinterpret_cast<__nv_bfloat16*>(v);
  ga.dst_rows = dst_rows;
  ga.max_rows = max_rows;
  ga.ready = p->ready;
  // (the time-out test hook: a count that no norm kernel will ever publish; the handle's own target stays)
  ga.ready_target = (int)(p->ready_target + (without_norm ? (unsigned)n_tokens : 0u));
  ga.wait_cycles = p->wait_cycles > 0 ? p->wait_cycles : Q_WAIT_CYCLES;
  ga.ws = p->ws;
  ga.counters = p->counters;
  ga.status = p->status;
  const int n_ctas = (int)std::min<long long>(p->num_sms, ga.total_chunks);
  ga.hp = 0;
  if (ga.tn <= 64 && n_ctas > ga.n_tiles && n_ctas < 2 * ga.n_tiles && !p->plain_split) {
    // closers take `per_closer` chunks each, helpers about HEAD_START chunks fewer
    const int HEAD_START = 8;
    const int n_helpers = n_ctas - ga.n_tiles;
    const long long num = ga.total_chunks + (long long)n_helpers * HEAD_START;
    const int per_closer = (int)((num + n_ctas - 1) / n_ctas);
    const int hp = ga.kc - per_closer;
    if (hp >= 1 && (long long)ga.n_tiles * hp >= n_helpers) ga.hp = hp;
  }

  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(n_ctas);
  cfg.blockDim = dim3(G_THREADS);
  cfg.dynamicSmemBytes = SMQ_TOTAL;
  cfg.stream = s;
  cfg.attrs = attr;
  cfg.numAttrs = no_pdl ? 0 : 1;
  if (p->ev_start && p->ev_stop) {
    cfg.numAttrs = 0;   // an event between the two kernels: an ordinary launch
    QCU_TRY(p, cudaEventRecord(p->ev_start, s));
  }
  if (ga.hp > 0) QCU_TRY(p, cudaLaunchKernelEx(&cfg, qkv_gemm_kernel<true>, p->w_map, p->x_map[tn_idx], ga));
  else QCU_TRY(p, cudaLaunchKernelEx(&cfg, qkv_gemm_kernel<false>, p->w_map, p->x_map[tn_idx], ga));
  if (p->ev_start && p->ev_stop) QCU_TRY(p, cudaEventRecord(p->ev_stop, s));
  p->last_launches++;
  return LACACHE_OK;
}
}  // namespace
}  // namespace lacache

extern "C" {

lacache_status lacache_qkv_set_wait_limit(lacache_qkv* p, double microseconds) {
  if (!p) return LACACHE_ERR_INVALID_ARG;
  if (!(microseconds >= 0.0) || microseconds > 1.0e7) return qfail(p, LACACHE_ERR_INVALID_ARG, "wait limit %g us", microseconds);
  p->wait_cycles = (long long)(microseconds * 2000.0);   // SM clock cycles at about 2 GHz
  return LACACHE_OK;
}

lacache_status lacache_qkv_project_without_norm(lacache_qkv* p, const void* hidden, int n_tokens, void* q, void* k,
                                                void* v, void* stream) {
  return lacache::project_impl(p, nullptr, hidden, n_tokens, q, k, v, nullptr, nullptr, 0, false, stream, true);
}

lacache_status lacache_qkv_set_timing_events(lacache_qkv* p, void* ev_start, void* ev_stop) {
  if (!p) return LACACHE_ERR_INVALID_ARG;
  p->ev_start = (cudaEvent_t)ev_start;
  p->ev_stop = (cudaEvent_t)ev_stop;
  return LACACHE_OK;
}

int lacache_qkv_last_launch_count(const lacache_qkv* p) { return p ? p->last_launches : -1; }

lacache_status lacache_qkv_poll_status(lacache_qkv* p) {
  if (!p) return LACACHE_ERR_INVALID_ARG;
  QCU_TRY(p, cudaDeviceSynchronize());
  int32_t w[4] = {0, 0, 0, 0};
  QCU_TRY(p, cudaMemcpy(w, p->status, 16, cudaMemcpyDeviceToHost));
  if (w[0] == 0) return LACACHE_OK;
  QCU_TRY(p, cudaMemset(p->status, 0, 16));
  if (w[1] == QLOC_TOKEN_ID)
    return qfail(p, (lacache_status)w[0], "token id %d of input row %d is outside the embedding table", w[3], w[2]);
  if (w[1] == QLOC_ROW)
    return qfail(p, (lacache_status)w[0], "destination row %d of input row %d is out of range", w[3], w[2]);
  return qfail(p, (lacache_status)w[0], "device status %d at location %d (block %d, thread %d)", w[0], w[1], w[2], w[3]);
}

const char* lacache_qkv_last_error(const lacache_qkv* p) { return p ? p->err : g_qkv_create_err; }

}  // extern "C"
