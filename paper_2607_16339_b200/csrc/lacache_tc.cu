// tcgen05 attention kernel for sm_100a (bf16 inputs, head_dim 128).
//
// One persistent CTA per SM, warp-specialised:
//   warp 0 (one lane)  producer: TMA loads of Q, K, V tiles into shared memory
//   warp 1 (one lane)  issues tcgen05.mma and commits completion to mbarriers
//   warps 2..9         256 "row" threads: TMEM lane r = query row r of the
//                      tile, two threads per row (each owns half of the
//                      columns / features)
//
// Arithmetic (Eq. 2-6 with base-2 exponentials):
//   S  = Q' K'^T   kind::f16 MMA on bf16 operands from shared memory, fp32
//                  accumulator in TMEM.  Rotated Q', K' are stored as
//                  hi + lo bf16 planes; S = hi.hi + hi.lo + lo.hi.
//   P~ = 2^(S c - m), m an INTEGER reference exponent (every rescale factor is
//                  an exact power of two), rounded to fp16, written to TMEM.
//   O~ = P~ V      MMA with A = P~ from TMEM, B = V (fp16, MN-major) from
//                  shared memory.  The normaliser sums the rounded P~.
//
// Two roles, chosen per CTA:
//   stream role  a tile of 128 (or 64) query rows streams key tiles of 128
//                keys; O~ accumulates in TMEM and is rescaled in place only
//                when a row maximum outgrows the reference exponent; used for the cache build
//                (rows in U x keys in U -> cached state), the full recompute,
//                and the block queries of a step (one chunk of key tiles per
//                work unit; the last chunk to finish merges the partials).
//   merge role   the reuse pass for fixed queries: per tile of 128 rows, the
//                scores against the block's keys, then
//                out = (alpha O~_cache + P~ V) / (alpha l_cache + sum P~).
//                O~_cache rows come in and out rows go out as bulk async
//                copies through a padded staging buffer, so all cache traffic
//                is coalesced and asynchronous.
// Every mbarrier wait is bounded; a wait that runs out sets the status word
// and the CTA unwinds (TMEM is always freed).
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <stdio.h>

#include "lacache_internal.h"
#include "lacache_ptx.h"
#include "lacache_rope_math.h"

namespace lacache {

struct TcMaps {
  // rotated Q' / K': 5-D views {64 features, Tp rows, 2 feature halves, heads, 2 planes (hi, lo)} of the
  // split-bf16 storage [plane][head][half][Tp][64]; one box = both planes and both halves of `rows` rows
  // of one head, laid out in shared memory as [plane][half][rows][64] (128-byte swizzle)
  alignas(64) CUtensorMap q;       // box 128 rows
  alignas(64) CUtensorMap q64;     // box 64 rows (block queries)
  // block queries of `pack` heads of one KV group side by side: dimensions ordered {64, rows, heads, halves,
  // planes}, box {64, pack_rows, pack, 2, 2}: lands as [plane][half][head][row][64], i.e. one 128-row tile
  alignas(64) CUtensorMap q_pack;
  alignas(64) CUtensorMap k;       // box TC_KEYS rows (stream role)
  alignas(64) CUtensorMap k64;     // box 64 rows (the block's keys, merge role)
  alignas(64) CUtensorMap k32;     // box 32 rows (the block's keys, pipelined merge role)
  // V: 4-D views {64, Tp, 2 halves, heads} of the fp16 storage [head][half][Tp][64]
  alignas(64) CUtensorMap v;
  alignas(64) CUtensorMap v64;
  alignas(64) CUtensorMap v32;
  alignas(64) CUtensorMap st_o;    // cached O~ [Hq][Tp][128] fp32, box 32 cols x 128 rows
  alignas(64) CUtensorMap out;     // caller's out [T][Hq][128] fp32, box 32 cols x 1 head x 128 rows
  alignas(64) CUtensorMap out_sub[4];  // the same with boxes of 64, 32, 16 and 8 rows (clipped row tiles)
  const void* out_ptr;             // the buffer `out` was encoded for
};

namespace {

constexpr int D = 128;
constexpr int BM = TC_ROWS;   // 128 query rows (TMEM lanes)
constexpr float RESCALE_SLACK = 3.f;
constexpr int ROW_WARPS = 8;
constexpr int ROW_THREADS = ROW_WARPS * 32;
constexpr int THREADS = 64 + ROW_THREADS + 32;   // warp 0: TMA producer, warp 1: MMA issuer, warps 2-9: row threads,
                                                  // warp 10: second MMA issuer (P~V products of the stream role)

// ---- shared memory map (bytes from a 1024-aligned base) ----
constexpr uint32_t SM_Q = 0;                      // Q hi plane (two boxes), then the lo plane
// stream role: two stages of one key tile {K hi (2 boxes), K lo (2 boxes)}, two stages of V
constexpr uint32_t SM_K = 65536;
constexpr uint32_t SM_XCH = 229376;   // both roles: 16 bytes per row for exchanges between the two threads of a row
// What depends on the precision mode.  SPLIT: rotated Q', K' as two bf16 planes (hi, lo), three score
// products, key tiles of 96 (two stages of keys AND of values fit beside the Q tile).  Plain: one plane,
// one product, key tiles of 128.
template <bool SPLIT>
struct Tile {
  static constexpr int BN = SPLIT ? TC_KEYS_SPLIT : TC_KEYS_PLAIN;   // keys per tile (stream role)
  static constexpr int HC = BN / 2;                                  // columns per row thread
  static constexpr uint32_t PLANES = SPLIT ? 2 : 1;
  static constexpr uint32_t KS_BOX = BN * 128;                       // one [BN rows][64 cols] 16-bit box
  static constexpr uint32_t K_STAGE = 2 * PLANES * KS_BOX;           // K hi (2 boxes) [, K lo (2 boxes)]
  static constexpr uint32_t SK_LO = 2 * KS_BOX;
  static constexpr uint32_t SM_V = SM_K + 2 * K_STAGE;               // two stages of V (2 boxes each)
  static constexpr uint32_t V_STAGE = 2 * KS_BOX;
  static_assert(BN % 32 == 0 && BN <= 128, "tile width");
  static_assert(KS_BOX % 1024 == 0, "swizzled boxes need 1024-byte alignment");
  static_assert(SM_V + 2 * V_STAGE <= SM_XCH, "stream-role tiles overrun");
  // (A key tile is wider than a block, so no tile lies wholly inside the keys a build excludes: every
  // tile in [t0, t1) is processed, excluded columns are masked by the row threads.)
  static_assert(BN > TC_MAX_BLOCK, "a key tile could fall wholly inside the excluded block");
};
// The stream role stages its epilogue (128 rows x 512 B, 16-byte chunks XOR-swizzled
// by the row so row-wise writes and row-wise reads are both conflict-free) in the
// Q region: in all of it for 128-row units (the next unit's Q load waits for the
// epilogue), in its upper half for 64-row units (whose Q tile needs only the lower half).
constexpr uint32_t STAGE_ROW = 512;
// paired step, one-plane operands: where the partner CTA puts its partial state -- O~ of up to 32 rows in the
// staging layout (512 bytes a row, 16-byte chunks XOR-swizzled by the row), then (m, l) per row
constexpr uint32_t SM_RX = Tile<false>::SM_V + 2 * Tile<false>::V_STAGE;
constexpr uint32_t SM_RX_ML = SM_RX + 32 * STAGE_ROW;
static_assert(SM_RX_ML + 32 * 8 <= SM_XCH, "no room for the partner's partial state");
// build, one-plane operands: staging of a unit's cached O~ tile for bulk tensor stores, four swizzled boxes of
// 32 features x 128 rows -- two in the upper half of the Q region (a one-plane Q tile needs the lower half),
// two in the 32 KB behind the value stages
__host__ __device__ constexpr uint32_t st_box(int cb) { return cb < 2 ? SM_Q + 32768u + (uint32_t)cb * 16384u : SM_RX + (uint32_t)(cb - 2) * 16384u; }
static_assert(SM_RX + 2 * 16384u <= SM_XCH, "no room for the state staging tile");
// merge role: the 96 KB after Q hold 2 stages of the block's keys {K hi, K lo, V} of 64
// rows, then the staging tile of the cached O~ / the output
constexpr uint32_t SM_KV = SM_K;
constexpr uint32_t KV_STAGE = 49152;
constexpr uint32_t KV_KLO = 16384;
constexpr uint32_t KV_V = 32768;
constexpr uint32_t K_BOX = 64 * 128;              // one [64 rows][64 cols] 16-bit box
constexpr uint32_t SM_IO = SM_KV + 2 * KV_STAGE;  // four swizzled boxes of 32 fp32 columns x 128 rows
constexpr uint32_t IO_BOX = 128 * 128;
static_assert(SM_IO + 4 * IO_BOX <= SM_XCH, "merge-role staging overruns");
constexpr uint32_t SM_BAR = SM_XCH + BM * 16;
constexpr uint32_t SM_TOTAL = SM_BAR + 256;
static_assert(SM_TOTAL <= 232448, "exceeds the 227 KB per-CTA limit");

// ---- TMEM columns ----
// merge role
constexpr uint32_t TM_S = 0;      // 2 x 64: scores
constexpr uint32_t TM_P = 128;    // 2 x 32: fp16 probabilities, two per column
constexpr uint32_t TM_O = 256;    // 2 x 128: P.V of one unit
// stream role
constexpr uint32_t TS_S = 0;      // 2 x 128 (BN used): scores
constexpr uint32_t TS_P = 256;    // 2 x 64 (BN/2 used): fp16 probabilities
constexpr uint32_t TS_O = 384;    // 128: O~ accumulated over the tiles of a unit
constexpr uint32_t TM_COLS = 512;

enum {
  BAR_Q_FULL = 0, BAR_Q_FREE,
  BAR_KV_FULL, BAR_KV_FULL1, BAR_KV_FREE, BAR_KV_FREE1,   // merge role: 2 stages
  BAR_K_FULL = BAR_KV_FULL, BAR_V_FULL = BAR_KV_FULL1,    // stream role: keys / values
  BAR_K_FREE = BAR_KV_FREE, BAR_V_FREE = BAR_KV_FREE1,
  BAR_S_FULL, BAR_S_FULL1, BAR_P_FULL, BAR_P_FULL1,
  BAR_O_FULL, BAR_O_FULL1, BAR_O_FREE, BAR_O_FREE1,
  BAR_IO_FULL, BAR_IO_FREE, BAR_EPI, BAR_DONE,
  BAR_K_FULL1, BAR_K_FREE1, BAR_V_FULL1, BAR_V_FREE1,  // stream role, second key / value stage
  BAR_QC,  // stream role: the row threads have written the rotated Q tile of the CTA's first unit
  BAR_IO_FULL1, BAR_OUT_RDY, BAR_OUT_RDY1,  // pipelined merge role: second staging tile; output tile b is complete
  BAR_PAIR,  // 4 barriers: the two warps that share a TMEM lane quadrant
  N_BARS = BAR_PAIR + 4,
  BAR_RX = BAR_IO_FULL,  // stream role of a paired step (it has no staging-tile barriers): the partner's partial state has arrived
  // stream role of a build with one-plane operands: a unit's state tile is staged / its bulk store has read the staging
  BAR_ST_RDY = BAR_OUT_RDY, BAR_ST_FREE = BAR_IO_FREE
};

enum { EPI_STATE = 0, EPI_OUT = 1, EPI_PARTIAL = 2, EPI_SEND = 3 };   // SEND: the partial state goes to the partner CTA

constexpr long long WAIT_CYCLES = 4000000000ll;  // ~2 s

using namespace ptx;

// both planes and both feature halves of `rows` rows of head h, starting at row `row`
__device__ __forceinline__ void load_qk_box(uint32_t dst, const CUtensorMap* map, uint32_t bar, int row, int h) {
  tma_load_5d(dst, map, bar, 0, row, 0, h, 0);
}
__device__ __forceinline__ void load_v_box(uint32_t dst, const CUtensorMap* map, uint32_t bar, int row, int h) {
  tma_load_4d(dst, map, bar, 0, row, 0, h);
}
// one 32-byte store of 8 words (the address is 32-byte aligned)
__device__ __forceinline__ void st_global_v8(void* dst, const uint32_t* r) {
  asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(dst), "r"(r[0]), "r"(r[1]), "r"(r[2]),
               "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7])
               : "memory");
}
// one 32-byte load of 8 words (the address is 32-byte aligned)
__device__ __forceinline__ void ld_global_v8(const void* src, uint32_t* r) {
  asm volatile("ld.global.v8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
               : "l"(src)
               : "memory");
}
__device__ __forceinline__ unsigned long long global_timer_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// p rounded to 11 significant bits (what fp16 keeps) with plain fp32 arithmetic
// (Veltkamp split), so the fp16 conversion that follows is exact and the
// normaliser can sum the very values the MMA multiplies without converting back.
__device__ __forceinline__ float round_to_half_bits(float p) {
  float c = __fmul_rn(p, 8193.0f);
  return __fsub_rn(c, __fsub_rn(c, p));
}
// four consecutive output elements at element offset `off` of `out` (fp32, or bf16 when the context's
// out_dtype says so)
__device__ __forceinline__ uint32_t pack_bf16x2(float a, float b) {
  __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&h);
}
__device__ __forceinline__ void store_out4(const AttnArgs& a, size_t off, float4 v) {
  if (a.out_bf16) {
    *reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(a.out) + off) =
        make_uint2(pack_bf16x2(v.x, v.y), pack_bf16x2(v.z, v.w));
  } else {
    *reinterpret_cast<float4*>(a.out + off) = v;
  }
}
__device__ __forceinline__ WorkItem load_item(const WorkItem* p) {
  const int4* q = reinterpret_cast<const int4*>(p);
  int4 a = __ldg(q), b = __ldg(q + 1), c = __ldg(q + 2);
  WorkItem w;
  w.kind = a.x; w.seq = a.y; w.row0 = a.z; w.nrows = a.w;
  w.chunk = b.x; w.kt0 = b.y; w.kt1 = b.z; w.pad = b.w;
  w.seq_start = c.x; w.seq_end = c.y; w.blk_start = c.z; w.pad2 = c.w;
  return w;
}



struct Cta {
  uint32_t base;            // shared-space address of the region
  uint8_t* gen;             // generic pointer to the same region
  uint32_t tmem;            // TMEM base address
  volatile int* abort_flag;
  volatile uint32_t* flag;  // scratch word for CTA-wide decisions
  int32_t* status;
  __device__ __forceinline__ uint32_t bar(int slot) const { return base + SM_BAR + 8u * slot; }
};

// Bounded wait on phase `parity`; false if it ran out or the CTA is unwinding.
__device__ __noinline__ bool wait_slow(const Cta& c, uint32_t bar, uint32_t parity, int loc) {
  long long t0 = clock64();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 32; ++i)
      if (mbar_try(bar, parity)) return true;
    if (*c.abort_flag) return false;
    if (clock64() - t0 > WAIT_CYCLES) {
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
__device__ __forceinline__ bool wait_bar(const Cta& c, int slot, uint32_t parity, int loc) {
  uint32_t b = c.bar(slot);
  if (mbar_try(b, parity)) return true;
  return wait_slow(c, b, parity, loc);
}

// One unit of work of the stream role, decoded identically by every warp role.
// What the stream role's templates are instantiated for: a build or a full recompute; a step; a build
// over key windows (units may start from a stored state and store a snapshot: the incremental rebuild).
// Separate kernels, so that the plain build and the step carry none of the window code.
// KIND_STEP2: a step whose block-row units all have exactly two key chunks, run by the two CTAs of a
// thread-block cluster: the CTA with the second chunk hands its partial state to its partner through
// distributed shared memory, and the partner writes the merged rows (one round of units, unpacked heads,
// one-plane operands: the receiving buffer needs 32 KB that the split planes' tiles leave no room for).
enum StreamKind : int { KIND_BUILD = 0, KIND_STEP = 1, KIND_WINDOW = 2, KIND_STEP2 = 3 };
__host__ __device__ constexpr bool kind_is_step(int k) { return k == KIND_STEP || k == KIND_STEP2; }

struct Unit {
  int row0, nrows, h, kh, seq;
  int key_base, t0, t1;   // key tiles [t0, t1): tile t holds keys key_base + 64 t ...
  int k0, k1, x0, x1;     // valid keys [k0, k1) minus [x0, x1)
  int epi, chunk, nchunks;
  int q_rows;             // rows of the Q box: 128 or 64
  int nh, rh;             // packed block queries: nh heads h, h + 1, ... of one KV group, rh lanes each (rh = 0: one head)
  int init;               // build over a key window: the unit starts from the rows' state in a.init instead of an empty one
  int snap;               // ... and stores the state it has after its first key tile to a.snap
  int base1;              // >= 0: key tiles after the first are counted from this token instead of key_base + BN
};
// first key (token index) of key tile t of a unit
template <int KIND, bool SPLIT>
__device__ __forceinline__ int tile_key_row(const Unit& un, int t) {
  constexpr int BN = Tile<SPLIT>::BN;
  if (KIND == KIND_WINDOW && un.base1 >= 0 && t > 0) return un.base1 + (t - 1) * BN;
  return un.key_base + t * BN;
}
// head and row within the head's rows of tile row r; whether r holds a real query row (rh is 0, 32 or 64)
__device__ __forceinline__ int unit_head(const Unit& un, int r) { return un.rh ? un.h + (r >> (un.rh == 64 ? 6 : 5)) : un.h; }
__device__ __forceinline__ int unit_row(const Unit& un, int r) { return un.rh ? (r & (un.rh - 1)) : r; }
__device__ __forceinline__ bool unit_row_valid(const Unit& un, int r) {
  return un.rh ? ((r >> (un.rh == 64 ? 6 : 5)) < un.nh && (r & (un.rh - 1)) < un.nrows) : r < un.nrows;
}

// which work item unit u belongs to (units are head-minor; in a paired step unit pair u / 2 is head
// (u / 2) % Hq of sequence (u / 2) / Hq, and u % 2 its key chunk: a sequence's two chunk items are adjacent)
template <bool PACKED, int KIND>
__device__ __forceinline__ int unit_item(const Geometry& g, const AttnArgs& a, int u) {
  if (KIND == KIND_STEP2) return ((u >> 1) / g.Hq) * 2 + (u & 1);
  return u / (PACKED ? a.stream_slots : g.Hq);
}

// PACKED (a.pack > 1): the units are block queries of several heads side by side in one tile.  A template
// parameter of the whole kernel, so that the kernel a build or an MHA step runs carries none of the per-row
// head arithmetic: this kernel is sensitive to its code size.
template <bool PACKED, int KIND, bool SPLIT>
__device__ __forceinline__ Unit decode_stream(const Geometry& g, const AttnArgs& a, const WorkItem& it, int u) {
  using TL = Tile<SPLIT>;
  constexpr int BN = TL::BN;
  constexpr bool STEP = kind_is_step(KIND);
  constexpr bool WINDOW = KIND == KIND_WINDOW;
  (void)WINDOW;
  Unit un;
  // units are head-minor: unit u = item u / slots of head (or head group) u % slots (a CTA's units, a
  // fixed stride apart, then cycle through the items instead of drawing one item's heads)
  const int slot = (KIND == KIND_STEP2 ? (u >> 1) : u) % (PACKED ? a.stream_slots : g.Hq);
  if (PACKED) {
    const int per_kv = (g.group + a.pack - 1) / a.pack;
    un.kh = slot / per_kv;
    const int s = slot % per_kv;
    un.h = un.kh * g.group + s * a.pack;
    un.nh = min(a.pack, g.group - s * a.pack);
    un.rh = a.pack_rows;
  } else {
    un.h = slot;
    un.kh = un.h / g.group;
    un.nh = 1;
    un.rh = 0;
  }
  un.seq = it.seq;
  un.row0 = it.row0;
  un.nrows = it.nrows;
  un.key_base = it.seq_start;
  un.k0 = it.seq_start;
  un.k1 = it.seq_end;
  un.x0 = un.x1 = 0;
  un.t0 = 0;
  un.t1 = (it.seq_end - it.seq_start + BN - 1) / BN;
  un.chunk = 0;
  un.nchunks = 1;
  un.q_rows = BM;
  un.init = un.snap = 0;
  un.base1 = -1;
  if (WINDOW) {
    // keys [kt0, kt1) of the sequence (token indices), optionally without the block's; tiles are
    // counted from token `pad`, which may lie before the window (and before token 0: those key rows
    // load as zeros and are masked like every key outside the window)
    un.key_base = it.pad;
    un.k0 = it.kt0;
    un.k1 = it.kt1;
    un.t1 = it.kt1 > it.pad ? (it.kt1 - it.pad + BN - 1) / BN : 0;
    if (it.chunk & 4) {
      un.x0 = it.blk_start;
      un.x1 = it.blk_start + g.block_len;
    }
    if (it.chunk & 8) {
      // the first tile ends where the block starts; the others start right after the block
      un.base1 = it.blk_start + g.block_len;
      un.t1 = 1 + (it.kt1 > un.base1 ? (it.kt1 - un.base1 + BN - 1) / BN : 0);
    }
    un.epi = (it.chunk & 16) ? EPI_OUT : EPI_STATE;   // bit 4: normalised rows to out / lse instead of a state
    un.init = it.chunk & 1;
    un.snap = (it.chunk >> 1) & 1;
  } else if (!STEP && a.mode == MODE_BUILD) {
    un.x0 = it.blk_start;
    un.x1 = it.blk_start + g.block_len;
    un.epi = EPI_STATE;
  } else if (STEP) {
    un.t0 = it.kt0;
    un.t1 = it.kt1;
    un.chunk = it.chunk;
    un.nchunks = it.pad;
    // (block rows whose result is a state, not normalised rows, always leave partial states: a launch of
    // its own merges them)
    un.epi = (it.pad > 1 || a.blk_to_state) ? EPI_PARTIAL : EPI_OUT;
    if (KIND == KIND_STEP2) un.epi = it.chunk == 0 ? EPI_OUT : EPI_SEND;   // (every unit has two chunks)
    un.q_rows = un.rh ? BM : 64;
  } else {
    un.epi = EPI_OUT;
  }
  return un;
}

// S (+)= Q' K'^T as hi.hi + hi.lo + lo.hi; Q planes at q_base (lo plane after the hi
// plane's two boxes) with boxes of q_box bytes, K planes at k_hi / k_lo with boxes of
// k_box bytes.  The four base descriptors are built once; each MMA adds a small
// constant to the start-address field (a single thread issues these back to back,
// so every instruction saved here shortens the critical path).
template <bool SPLIT>
__device__ __forceinline__ void issue_s_mma(uint32_t q_base, uint32_t q_box, uint32_t k_hi, uint32_t k_lo,
                                            uint32_t k_box, uint32_t s_tmem, uint32_t idesc) {
  const uint64_t qd[2] = {smem_desc(q_base, 16, 1024), smem_desc(q_base + 2u * q_box, 16, 1024)};
  const uint64_t kd[2] = {smem_desc(k_hi, 16, 1024), smem_desc(k_lo, 16, 1024)};
  const uint32_t qb16 = q_box >> 4, kb16 = k_box >> 4;
  uint32_t acc = 0;
#pragma unroll
  for (int term = 0; term < (SPLIT ? 3 : 1); ++term) {   // hi.hi [+ hi.lo + lo.hi]
    const uint64_t qa = qd[term == 2 ? 1 : 0];
    const uint64_t ka = kd[term == 1 ? 1 : 0];
#pragma unroll
    for (int ks = 0; ks < D / 16; ++ks) {
      const uint32_t qoff = (ks >> 2) * qb16 + (ks & 3) * 2;
      const uint32_t koff = (ks >> 2) * kb16 + (ks & 3) * 2;
      mma_ss(s_tmem, qa + qoff, ka + koff, idesc, acc);
      acc = 1;
    }
  }
}
// O (+)= P~ V: A = P~ in TMEM (16 keys = 8 columns per step), B = V tile, MN-major:
// 64 features contiguous (128 B), the next 64 features v_box bytes further (LBO),
// groups of 8 keys 1 KB apart (SBO); 16 keys = 2 KB.
__device__ __forceinline__ void issue_pv_mma(uint32_t v_base, uint32_t v_box, uint32_t p_tmem, uint32_t o_tmem,
                                             int ksteps, uint32_t accumulate) {
  constexpr uint32_t idesc = idesc_f16(0u /*fp16*/, 1u, BM, D);
  const uint64_t vd = smem_desc(v_base, v_box, 1024);
  for (int ks = 0; ks < ksteps; ++ks)
    mma_ts(o_tmem, p_tmem + 8 * ks, vd + (uint64_t)(ks * (2048 >> 4)), idesc, (ks > 0) ? 1u : accumulate);
}
template <bool SPLIT>
__device__ __forceinline__ void load_kv_tile(const TcMaps& maps, uint32_t kv_base, uint32_t bar, int krow, int kh) {
  static_assert(KV_KLO == 2 * K_BOX && KV_V == 4 * K_BOX, "K hi, K lo and V boxes are contiguous");
  mbar_expect_tx(bar, (SPLIT ? 6 : 4) * K_BOX);   // (one plane: the place of the lo boxes stays empty)
  load_qk_box(kv_base, &maps.k64, bar, krow, kh);
  load_v_box(kv_base + KV_V, &maps.v64, bar, krow, kh);
}
template <bool SPLIT>
__device__ __forceinline__ void load_q_tile(const Cta& c, const TcMaps& maps, int q_rows, int row0, int h,
                                            bool packed = false) {
  const uint32_t bar = c.bar(BAR_Q_FULL);
  const uint32_t box = (uint32_t)q_rows * 128u;
  mbar_expect_tx(bar, (SPLIT ? 4 : 2) * box);
  if (packed) tma_load_5d(c.base + SM_Q, &maps.q_pack, bar, 0, row0, h, 0, 0);   // heads h, h + 1, ... side by side
  else load_qk_box(c.base + SM_Q, q_rows == 64 ? &maps.q64 : &maps.q, bar, row0, h);
}

// ===========================================================================
// stream role
// ===========================================================================
// The producer walks the (unit, tile) sequence twice, with independent cursors for
// keys (with the unit's Q tile) and for values, and issues whichever load has a
// free stage: waiting for a value stage must not hold back the next key tile.
struct TileCursor {
  int u, uu, t, jj;   // unit index, ordinal of the unit in this CTA, tile, global tile ordinal
  WorkItem it;
  Unit un;
  bool valid, q_done, loads_q;
};
template <bool PACKED, int KIND, bool SPLIT>
__device__ __forceinline__ void cursor_load_unit(const Geometry& g, const AttnArgs& a, TileCursor& cu, int n_units) {
  constexpr bool STEP = kind_is_step(KIND);
  constexpr bool WINDOW = KIND == KIND_WINDOW;
  (void)WINDOW;
  cu.valid = cu.u < n_units;
  if (!cu.valid) return;
  cu.it = load_item(a.items + unit_item<PACKED, KIND>(g, a, cu.u));
  cu.un = decode_stream<PACKED, KIND, SPLIT>(g, a, cu.it, cu.u);
  cu.t = cu.un.t0;
  cu.q_done = !cu.loads_q;
}
template <bool PACKED, int KIND, bool SPLIT>
__device__ __forceinline__ void cursor_advance(const Geometry& g, const AttnArgs& a, TileCursor& cu, int stride,
                                               int n_units) {
  constexpr bool STEP = kind_is_step(KIND);
  constexpr bool WINDOW = KIND == KIND_WINDOW;
  (void)WINDOW;
  // move to the next tile; cross into the next unit(s) when this one is exhausted
  if (cu.t < cu.un.t1) {
    ++cu.t;
    ++cu.jj;
  }
  while (cu.valid && cu.t >= cu.un.t1 && cu.q_done) {
    cu.u += stride;
    ++cu.uu;
    cursor_load_unit<PACKED, KIND, SPLIT>(g, a, cu, n_units);
  }
}

template <bool PACKED, int KIND, bool SPLIT>
__device__ void stream_producer(const Cta& c, const TcMaps& maps, const Geometry& g, const AttnArgs& a,
                                int first, int stride, int n_units, WorkItem it) {
  using TL = Tile<SPLIT>;
  constexpr int BN = TL::BN;
  constexpr uint32_t KS_BOX = TL::KS_BOX, K_STAGE = TL::K_STAGE, SM_V = TL::SM_V, V_STAGE = TL::V_STAGE;
  constexpr bool STEP = kind_is_step(KIND);
  constexpr bool WINDOW = KIND == KIND_WINDOW;
  (void)WINDOW;
  // three independent cursors: Q tiles (one per unit), key tiles, value tiles
  TileCursor cq, ck, cv;
  cq.u = first; cq.uu = 0; cq.jj = 0; cq.loads_q = true;
  cursor_load_unit<PACKED, KIND, SPLIT>(g, a, cq, n_units);
  ck = cq;
  ck.loads_q = false;  // the key and value cursors never load Q
  ck.q_done = true;
  if (ck.valid && ck.t >= ck.un.t1) cursor_advance<PACKED, KIND, SPLIT>(g, a, ck, stride, n_units);
  cv = ck;
  // What the RoPE kernel launched just before this one writes must not be loaded
  // before that grid has completed (this kernel may have started early): in a step
  // that is the block's rows -- every Q tile of this role and the key/value tiles
  // that overlap the block -- so tiles of fixed tokens are requested at once and
  // the wait comes only when nothing else can be issued.
  bool dep_done = false;
  // build with one-plane operands: full row tiles leave as bulk tensor stores from a staging tile the row
  // threads fill (units in the order of the Q loads; at most two are between their Q load and their store)
  constexpr bool STAGED = KIND == KIND_BUILD && !SPLIT;
  int st_slot0 = 0, st_slot1 = 0;   // row0 | head << 24 of the (at most two) units between their Q load and their store
  int st_head = 0, st_tail = 0;
  bool st_pending = false;
  const bool q_computed = STEP && a.q_raw != nullptr;
  auto tile_depends = [&](const TileCursor& cu) {
    if (!STEP) return true;
    const int krow = cu.un.key_base + cu.t * BN;
    return krow < cu.it.blk_start + g.block_len && krow + BN > cu.it.blk_start;
  };
  long long t_idle = 0;
  while (cq.valid || ck.valid || cv.valid || (STAGED && (st_head < st_tail || st_pending))) {
    bool did = false, blocked_on_dep = false;
    if (STAGED && st_head < st_tail && mbar_test(c.bar(BAR_ST_RDY), st_head & 1)) {
      // (dep_done: the unit's Q tile was loaded after the wait for the preceding grids, so no store precedes it)
      const int sv = (st_head & 1) ? st_slot1 : st_slot0;
      if (sv >= 0) {
#pragma unroll
        for (int cb = 0; cb < 4; ++cb) tma_store_3d(&maps.st_o, c.base + st_box(cb), 32 * cb, sv & 0xFFFFFF, sv >> 24);
        bulk_commit();
        st_pending = true;
      } else {
        mbar_arrive(c.bar(BAR_ST_FREE));
      }
      ++st_head;
      did = true;
    }
    if (cq.valid) {  // a unit without key tiles still needs its Q load (the MMA thread waits for it)
      if (cq.uu == 0 && q_computed) {
        // the row threads rotate this tile from the raw queries: nothing to load,
        // nothing to wait for (the plain arrival keeps the barrier's phase count in step)
        mbar_arrive(c.bar(BAR_Q_FULL));
        cq.q_done = true;
        cq.t = cq.un.t1;
        cursor_advance<PACKED, KIND, SPLIT>(g, a, cq, stride, n_units);
        did = true;
      } else if (!dep_done) {
        blocked_on_dep = true;
      } else if (cq.uu == 0 || mbar_test(c.bar(BAR_Q_FREE), (cq.uu - 1) & 1)) {
        load_q_tile<SPLIT>(c, maps, cq.un.q_rows, cq.un.row0, cq.un.h, cq.un.rh != 0);
        if (STAGED && a.st_tma && cq.un.epi == EPI_STATE) {
          const int sv = cq.un.row0 | (cq.un.h << 24) | (cq.un.nrows == BM ? 0 : (int)0x80000000u);   // (top bit: a clipped tile, nothing staged)
          if (st_tail & 1) st_slot1 = sv; else st_slot0 = sv;
          ++st_tail;
        }
        cq.q_done = true;
        cq.t = cq.un.t1;
        cursor_advance<PACKED, KIND, SPLIT>(g, a, cq, stride, n_units);
        // a build's Q tiles come from HBM once the batch outgrows L2: the next unit's tile is asked
        // into L2 a whole unit ahead of its load
        if (!STEP && cq.valid) tma_prefetch_5d(&maps.q, 0, cq.un.row0, 0, cq.un.h, 0);
        did = true;
      }
    }
    if (ck.valid && ck.t < ck.un.t1) {
      const int sk = ck.jj & 1, kuse = ck.jj >> 1;
      if (!dep_done && tile_depends(ck)) {
        blocked_on_dep = true;
      } else if (kuse == 0 || mbar_test(c.bar(sk ? BAR_K_FREE1 : BAR_K_FREE), (kuse - 1) & 1)) {
        const int krow = tile_key_row<KIND, SPLIT>(ck.un, ck.t);
        const uint32_t bar = c.bar(sk ? BAR_K_FULL1 : BAR_K_FULL);
        const uint32_t khi = c.base + SM_K + sk * K_STAGE;
        mbar_expect_tx(bar, K_STAGE);
        load_qk_box(khi, &maps.k, bar, krow, ck.un.kh);  // (split: the lo plane lands at khi + SK_LO)
        cursor_advance<PACKED, KIND, SPLIT>(g, a, ck, stride, n_units);
        did = true;
      }
    }
    if (cv.valid && cv.t < cv.un.t1) {
      const int sv = cv.jj & 1, vuse = cv.jj >> 1;
      if (!dep_done && tile_depends(cv)) {
        blocked_on_dep = true;
      } else if (vuse == 0 || mbar_test(c.bar(sv ? BAR_V_FREE1 : BAR_V_FREE), (vuse - 1) & 1)) {
        const int krow = tile_key_row<KIND, SPLIT>(cv.un, cv.t);
        const uint32_t bar = c.bar(sv ? BAR_V_FULL1 : BAR_V_FULL), vb = c.base + SM_V + sv * V_STAGE;
        mbar_expect_tx(bar, 2 * KS_BOX);
        load_v_box(vb, &maps.v, bar, krow, cv.un.kh);
        cursor_advance<PACKED, KIND, SPLIT>(g, a, cv, stride, n_units);
        did = true;
      }
    }
    if (!did && blocked_on_dep) {
      grid_dependency_wait();
      dep_done = true;
      did = true;
    }
    if (STAGED && !did && st_pending) {   // nothing else to issue: the last store has read its staging tile by now
      bulk_wait_read();
      mbar_arrive(c.bar(BAR_ST_FREE));
      st_pending = false;
      did = true;
    }
    if (did) {
      t_idle = 0;
    } else {  // nothing free: bounded idle
      if (t_idle == 0) t_idle = clock64();
      if (*c.abort_flag) break;
      if (clock64() - t_idle > WAIT_CYCLES) {
        *c.abort_flag = 1;
        if (atomicCAS(c.status, 0, (int)LACACHE_ERR_TIMEOUT) == 0) {
          c.status[1] = LOC_WAIT_K; c.status[2] = blockIdx.x; c.status[3] = threadIdx.x;
        }
        break;
      }
    }
  }
  if (STAGED) bulk_wait_read();  // shared memory stays valid until the last store has read it
  // (a CTA without units never touches memory the RoPE kernel writes)
}

// Two threads issue the stream role's MMAs, each a fixed pipeline with blocking (bounded) waits: one
// the score products, the other the P~V products.  tcgen05.mma accepts the next instruction only when the
// tensor pipe has room, so a single issuer leaves the pipe idle while it runs the scalar code between two
// batches (barrier waits, commits); with two issuers one thread's bookkeeping overlaps the other's MMAs.
// Scores of tile j need its keys and the score buffer of tile j - 2 read (= the probabilities of tile
// j - 2 written); P~V of tile j needs its probabilities and its values.  Each code block exists once
// (the unrolled MMA sequences are large, and cold instruction fetches are slow).
template <bool PACKED, int KIND, bool SPLIT>
__device__ void stream_mma_scores(const Cta& c, const Geometry& g, const AttnArgs& a, int first, int stride,
                                  int n_units, WorkItem it) {
  using TL = Tile<SPLIT>;
  constexpr int BN = TL::BN;
  constexpr uint32_t KS_BOX = TL::KS_BOX, K_STAGE = TL::K_STAGE, SK_LO = TL::SK_LO;
  constexpr bool STEP = kind_is_step(KIND);
  constexpr bool WINDOW = KIND == KIND_WINDOW;
  (void)WINDOW;
  // (operand format of the score product: bf16 planes, or fp16 in the one-plane fp16 mode)
  const uint32_t IDESC_S = idesc_f16((!SPLIT && g.op_f16) ? 0u : 1u, 0u, BM, BN);
  int uu = 0;
  uint32_t js = 0;  // score tiles issued so far (stage and buffer = js & 1, phase = (js >> 1) & 1)
  for (int u = first; u < n_units; u += stride, ++uu) {
    WorkItem nxt = it;
    if (u + stride < n_units) nxt = load_item(a.items + unit_item<PACKED, KIND>(g, a, u + stride));
    const Unit un = decode_stream<PACKED, KIND, SPLIT>(g, a, it, u);
    const uint32_t q_box = (uint32_t)un.q_rows * 128u;
    const int n_tiles = un.t1 - un.t0;
    if (!wait_bar(c, BAR_Q_FULL, uu & 1, LOC_WAIT_Q)) return;
    if (uu == 0 && STEP && a.q_raw != nullptr && !wait_bar(c, BAR_QC, 0, LOC_WAIT_Q)) return;
    for (int j = 0; j < n_tiles; ++j, ++js) {
      const uint32_t sk = js & 1u, b = js & 1u;
      // the score buffer was last used two tiles ago (possibly by the previous unit): its
      // probabilities have been written, so its scores have been read
      if (js >= 2 && !wait_bar(c, BAR_P_FULL + b, ((js - 2) >> 1) & 1u, LOC_WAIT_S)) return;
      if (!wait_bar(c, sk ? BAR_K_FULL1 : BAR_K_FULL, (js >> 1) & 1u, LOC_WAIT_K)) return;
      const uint32_t khi = c.base + SM_K + sk * K_STAGE, klo = khi + SK_LO;
      tc_fence_after();
      issue_s_mma<SPLIT>(c.base + SM_Q, q_box, khi, klo, KS_BOX, c.tmem + TS_S + 128 * b, IDESC_S);
      tc_commit(c.bar(BAR_S_FULL + b));
      tc_commit(c.bar(sk ? BAR_K_FREE1 : BAR_K_FREE));
    }
    tc_commit(c.bar(BAR_Q_FREE));  // every score MMA of this unit has been issued (or it had no key tiles)
    it = nxt;
  }
}

template <bool PACKED, int KIND, bool SPLIT>
__device__ void stream_mma_pv(const Cta& c, const Geometry& g, const AttnArgs& a, int first, int stride,
                              int n_units, WorkItem it) {
  using TL = Tile<SPLIT>;
  constexpr int BN = TL::BN;
  constexpr uint32_t KS_BOX = TL::KS_BOX, SM_V = TL::SM_V, V_STAGE = TL::V_STAGE;
  constexpr bool STEP = kind_is_step(KIND);
  constexpr bool WINDOW = KIND == KIND_WINDOW;
  (void)WINDOW;
  int uu = 0;
  uint32_t jp = 0;  // P~V tiles issued so far
  for (int u = first; u < n_units; u += stride, ++uu) {
    WorkItem nxt = it;
    if (u + stride < n_units) nxt = load_item(a.items + unit_item<PACKED, KIND>(g, a, u + stride));
    const Unit un = decode_stream<PACKED, KIND, SPLIT>(g, a, it, u);
    const int n_tiles = un.t1 - un.t0;
    // O~ of the previous unit has been read by the row threads.  (A unit without key tiles issues nothing
    // and does not wait: the row threads cannot complete this unit's phase of the barrier before the
    // products of its tiles are done, so when a unit with tiles looks, the barrier is at most one phase on.)
    if (uu >= 1 && n_tiles > 0 && !wait_bar(c, BAR_O_FREE, (uu - 1) & 1, LOC_WAIT_O)) return;
    for (int j = 0; j < n_tiles; ++j, ++jp) {
      const uint32_t b = jp & 1u, sv = jp & 1u, ph = (jp >> 1) & 1u;
      if (!wait_bar(c, BAR_P_FULL + b, ph, LOC_WAIT_S)) return;
      if (!wait_bar(c, sv ? BAR_V_FULL1 : BAR_V_FULL, ph, LOC_WAIT_V)) return;
      tc_fence_after();
      issue_pv_mma(c.base + SM_V + sv * V_STAGE, KS_BOX, c.tmem + TS_P + 64 * b, c.tmem + TS_O, BN / 16,
                   (j == 0 && !(WINDOW && un.init)) ? 0u : 1u);
      tc_commit(c.bar(BAR_O_FULL));
      tc_commit(c.bar(sv ? BAR_V_FREE1 : BAR_V_FREE));
    }
    it = nxt;
  }
}

// CTA-wide rendezvous of the row threads (bounded)
__device__ __forceinline__ bool epi_sync(const Cta& c, uint32_t& phase) {
  mbar_arrive(c.bar(BAR_EPI));
  bool ok = wait_bar(c, BAR_EPI, phase & 1, LOC_WAIT_O);
  ++phase;
  return ok;
}

// Cooperative, fully coalesced copy of the first nrows staging rows (512 B each,
// chunks XOR-swizzled by the row) to rows of `stride` floats in global memory:
// every warp-wide store writes one whole row.
__device__ __forceinline__ void coop_store_rows(const Cta& c, uint32_t stage_off, float* gbase, size_t stride,
                                                int nrows) {
  const int t = threadIdx.x - 64;
  for (int i = t; i < nrows * 32; i += ROW_THREADS) {
    const int rr = i >> 5, ch = i & 31;
    float4 v = *reinterpret_cast<const float4*>(c.gen + stage_off + rr * STAGE_ROW + ((ch ^ (rr & 7)) << 4));
    *reinterpret_cast<float4*>(gbase + (size_t)rr * stride + ch * 4) = v;
  }
}

// The same for rows of `out` (element offset `off0` of the first row, `stride` elements between rows), in
// the output's element type.
__device__ __forceinline__ void coop_store_out_rows(const Cta& c, const AttnArgs& a, uint32_t stage_off, size_t off0,
                                                    size_t stride, int nrows) {
  const int t = threadIdx.x - 64;
  for (int i = t; i < nrows * 32; i += ROW_THREADS) {
    const int rr = i >> 5, ch = i & 31;
    float4 v = *reinterpret_cast<const float4*>(c.gen + stage_off + rr * STAGE_ROW + ((ch ^ (rr & 7)) << 4));
    store_out4(a, off0 + (size_t)rr * stride + ch * 4, v);
  }
}

// Few chunks (at most NC): each thread takes BATCH (row, 16-byte column) items at a
// time and issues every load of the batch -- references, normalisers, 16 bytes of
// each partial O~ -- before any is used: one L2 round trip per batch.
template <int NC, int BATCH>
__device__ __forceinline__ void merge_few(const Geometry& g, const AttnArgs& a, size_t pbase, int nchunks,
                                          int block_len, int row0, int h) {
  const float LN2 = 0.69314718055994530942f;
  const int t = threadIdx.x - 64;
  const int n_items = block_len * 32;
  for (int i0 = t; i0 < n_items; i0 += BATCH * ROW_THREADS) {
    float mv[BATCH][NC], lv[BATCH][NC];
    float4 v[BATCH][NC];
#pragma unroll
    for (int bi = 0; bi < BATCH; ++bi) {
      const int i = min(i0 + bi * ROW_THREADS, n_items - 1);
      const int rr = i >> 5, ch = i & 31;
#pragma unroll
      for (int k = 0; k < NC; ++k) {
        const size_t pr = (pbase + min(k, nchunks - 1)) * block_len + rr;
        mv[bi][k] = __ldcg(a.part_m + pr);
        lv[bi][k] = __ldcg(a.part_l + pr);
        v[bi][k] = __ldcg(reinterpret_cast<const float4*>(a.part_o + pr * D) + ch);
      }
    }
#pragma unroll
    for (int bi = 0; bi < BATCH; ++bi) {
      const int i = i0 + bi * ROW_THREADS;
      if (i >= n_items) break;
      const int rr = i >> 5, ch = i & 31;
      float M = -INFINITY;
#pragma unroll
      for (int k = 0; k < NC; ++k)
        if (k < nchunks) M = fmaxf(M, mv[bi][k]);
      float L = 0.f;
      float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int k = 0; k < NC; ++k) {
        const float w = (k < nchunks && mv[bi][k] != -INFINITY) ? ex2(mv[bi][k] - M) : 0.f;
        L = fmaf(lv[bi][k], w, L);
        acc.x = fmaf(v[bi][k].x, w, acc.x);
        acc.y = fmaf(v[bi][k].y, w, acc.y);
        acc.z = fmaf(v[bi][k].z, w, acc.z);
        acc.w = fmaf(v[bi][k].w, w, acc.w);
      }
      const float inv = 1.f / L;
      const size_t orow = (size_t)(row0 + rr) * g.Hq + h;
      store_out4(a, orow * D + ch * 4, make_float4(acc.x * inv, acc.y * inv, acc.z * inv, acc.w * inv));
      if (ch == 0 && a.lse) a.lse[orow] = (M + log2f(L)) * LN2;
    }
  }
}

// Merge of the partial states of all key chunks of one (sequence, head) by the
// last chunk to arrive: thread t owns 16 bytes of one row; the partial rows are
// read with coalesced loads straight from L2 and the normalised rows written out.
__device__ __forceinline__ void merge_partials(const Geometry& g, const AttnArgs& a, size_t pbase, int nchunks,
                                               int block_len, int row0, int h) {
  const float LN2 = 0.69314718055994530942f;
  const int t = threadIdx.x - 64;
  if (nchunks <= 2) {
    merge_few<2, 4>(g, a, pbase, nchunks, block_len, row0, h);
    return;
  }
  if (nchunks <= 4) {
    merge_few<4, 2>(g, a, pbase, nchunks, block_len, row0, h);
    return;
  }
  for (int i = t; i < block_len * 32; i += ROW_THREADS) {
    const int rr = i >> 5, ch = i & 31;
    float M = -INFINITY;
    {
      float mv[16];  // at most 16 chunks: all loads in flight together
#pragma unroll
      for (int cc = 0; cc < 16; ++cc) mv[cc] = __ldcg(a.part_m + (pbase + min(cc, nchunks - 1)) * block_len + rr);
#pragma unroll
      for (int cc = 0; cc < 16; ++cc) M = fmaxf(M, mv[cc]);
    }
    float L = 0.f;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int c0 = 0; c0 < nchunks; c0 += 4) {
      float w[4];
      float4 v[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const int cc = min(c0 + k, nchunks - 1);
        const size_t pr = (pbase + cc) * block_len + rr;
        const float mcv = __ldcg(a.part_m + pr);
        w[k] = (c0 + k < nchunks && mcv != -INFINITY) ? ex2(mcv - M) : 0.f;
        L = fmaf(__ldcg(a.part_l + pr), w[k], L);
        v[k] = __ldcg(reinterpret_cast<const float4*>(a.part_o + pr * D) + ch);
      }
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        acc.x = fmaf(v[k].x, w[k], acc.x);
        acc.y = fmaf(v[k].y, w[k], acc.y);
        acc.z = fmaf(v[k].z, w[k], acc.z);
        acc.w = fmaf(v[k].w, w[k], acc.w);
      }
    }
    const float inv = 1.f / L;
    const size_t orow = (size_t)(row0 + rr) * g.Hq + h;
    store_out4(a, orow * D + ch * 4, make_float4(acc.x * inv, acc.y * inv, acc.z * inv, acc.w * inv));
    if (ch == 0 && a.lse) a.lse[orow] = (M + log2f(L)) * LN2;
  }
}

template <bool PACKED, int KIND, bool SPLIT>
__device__ void stream_rows(const Cta& c, const Geometry& g, const AttnArgs& a, int first, int stride, int n_units,
                            WorkItem it) {
  using TL = Tile<SPLIT>;
  constexpr int BN = TL::BN;
  constexpr int HC = TL::HC;
  constexpr bool STEP = kind_is_step(KIND);
  constexpr bool WINDOW = KIND == KIND_WINDOW;
  (void)WINDOW;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int quad = warp & 3;
  const int half = (warp - 2) >> 2;         // 0: first 64 columns / features, 1: the rest
  const int r = quad * 32 + lane;           // row of the tile = TMEM lane
  const uint32_t tlane = c.tmem + ((uint32_t)(quad * 32) << 16);
  const float LN2 = 0.69314718055994530942f;
  volatile float* xch = reinterpret_cast<volatile float*>(c.gen + SM_XCH + r * 16);  // 4 exchange slots per row
  uint32_t epi_phase = 0, epi_unit = 0, pair_phase = 0, xslot = 0;
  int jj = 0;
  int uu = -1;   // ordinal of the unit in this CTA
  for (int u = first; u < n_units; u += stride) {
    ++uu;
    WorkItem nxt = it;
    if (u + stride < n_units) nxt = load_item(a.items + unit_item<PACKED, KIND>(g, a, u + stride));
    const Unit un = decode_stream<PACKED, KIND, SPLIT>(g, a, it, u);
    it = nxt;
    if (u == first && STEP && a.q_raw != nullptr) {
      // The CTA's first unit: rotate the block's queries of this (sequence, head) here,
      // with the very arithmetic of the RoPE kernel, and write them where the TMA load
      // would have put them ([plane][feature half][row][64], 16-byte chunks XOR-swizzled
      // by the row), so this unit does not wait for that kernel.
      const int tq = threadIdx.x - 64;
      const uint32_t box = (uint32_t)un.q_rows * 128u;
      const int tile_rows = PACKED ? un.nh * un.rh : un.nrows;
      for (int i = tq; i < tile_rows * 8; i += ROW_THREADS) {
        const int qi = i >> 3, ch = i & 7, c0 = ch * 8;
        if (PACKED && !unit_row_valid(un, qi)) continue;   // lanes between a short block and the next head's rows
        const size_t src = (size_t)un.seq * g.block_len + unit_row(un, qi);   // row of the block's inputs
        const size_t soff = (src * g.Hq + unit_head(un, qi)) * D;
        float x1[8], x2[8], cs[8], sn[8], y1[8], y2[8];
        rope_load8(a.q_raw, soff + c0, true, x1);
        rope_load8(a.q_raw, soff + c0 + D / 2, true, x2);
        const float4* cp = reinterpret_cast<const float4*>(a.row_cos + src * (D / 2) + c0);
        const float4* sp = reinterpret_cast<const float4*>(a.row_sin + src * (D / 2) + c0);
        const float4 ca = cp[0], cb = cp[1], sa = sp[0], sb = sp[1];
        cs[0] = ca.x; cs[1] = ca.y; cs[2] = ca.z; cs[3] = ca.w; cs[4] = cb.x; cs[5] = cb.y; cs[6] = cb.z; cs[7] = cb.w;
        sn[0] = sa.x; sn[1] = sa.y; sn[2] = sa.z; sn[3] = sa.w; sn[4] = sb.x; sn[5] = sb.y; sn[6] = sb.z; sn[7] = sb.w;
        rope_rotate8(x1, x2, cs, sn, y1, y2);
        uint4 h1, l1, h2, l2;
        if (!SPLIT && g.op_f16) {
          h1 = rope_half8(y1);
          h2 = rope_half8(y2);
        } else {
          rope_split8(y1, h1, l1);
          rope_split8(y2, h2, l2);
        }
        uint8_t* const q0 = c.gen + SM_Q + qi * 128 + ((ch ^ (qi & 7)) << 4);
        *reinterpret_cast<uint4*>(q0) = h1;                 // hi plane, features [0, 64)
        *reinterpret_cast<uint4*>(q0 + box) = h2;           // hi plane, features [64, 128)
        if (SPLIT) {
          *reinterpret_cast<uint4*>(q0 + 2 * box) = l1;     // lo plane
          *reinterpret_cast<uint4*>(q0 + 3 * box) = l2;
        }
      }
      fence_async_smem();  // the MMA reads shared memory through the async proxy
      mbar_arrive(c.bar(BAR_QC));
    }
    const int row = un.row0 + unit_row(un, r);   // token of this tile row
    const int hrow = unit_head(un, r);           // and its query head
    const bool row_valid = unit_row_valid(un, r);
    const bool active = unit_row_valid(un, quad * 32);  // this warp holds at least one real row (its first)
    float m_ref = -INFINITY, l_part = 0.f;
    bool first_tile = true;
    bool calm = false;     // the unit's latest tile moved no reference exponent of this warp
    bool have_o = false;   // O~ in TMEM holds something before the unit's first P~V
    if (WINDOW && un.t1 <= un.t0) {
      // A unit without key tiles gives these threads nothing to wait for, and the other roles' parity
      // waits hold only while nobody runs more than one phase ahead: stay in step with the producer (the
      // unit's Q load lands only after the previous unit has been released by these threads).
      if (!wait_bar(c, BAR_Q_FULL, uu & 1, LOC_WAIT_Q)) return;
    }
    if (WINDOW && un.init) {
      // (the state may have been written by the launch just before this one)
      grid_dependency_wait();
      // The unit continues from a stored state (m, l, O~) of its rows: the reference exponent and the
      // normaliser go to registers (the normaliser to the first thread of the pair), O~ to the
      // accumulator columns this thread owns.  Nobody else reads or writes those cells between units
      // (the previous unit's P~V products are complete, and its epilogue read them from this thread).
      // The TMEM stores are warp-wide: rows past the end of a clipped tile store zeros.
      const size_t srow = (size_t)un.h * g.Tp + row;
      if (row_valid) {
        m_ref = a.init.m[srow];
        if (half == 0) l_part = a.init.l[srow];
      }
      const float4* src = reinterpret_cast<const float4*>(a.init.o + srow * D + 64 * half);
      {
        // all sixteen loads of the row half are in flight together (one round trip, not four)
        // (32-byte loads: a warp's load touches 32 rows whatever its width, so wider loads mean
        // fewer passes through the L1 tags; plain loads, not the read-only path: the launch may update
        // these rows in place)
        uint32_t rr[64];
#pragma unroll
        for (int i = 0; i < 64; ++i) rr[i] = 0u;
        if (row_valid) {
#pragma unroll
          for (int i = 0; i < 8; ++i) ld_global_v8(src + 2 * i, rr + 8 * i);
        }
        tmem_st32(tlane + TS_O + 64 * half, *reinterpret_cast<uint32_t(*)[32]>(rr));
        tmem_st32(tlane + TS_O + 64 * half + 32, *reinterpret_cast<uint32_t(*)[32]>(rr + 32));
      }
      tmem_st_wait();
      have_o = true;
      if (u + stride < n_units && (it.chunk & 1) && r < it.nrows) {
        // the next unit's rows of that state, asked into L2 now (`it` already holds its item)
        const char* nx = reinterpret_cast<const char*>(
            a.init.o + ((size_t)((u + stride) % g.Hq) * g.Tp + it.row0 + r) * D + 64 * half);
        prefetch_l2(nx);
        prefetch_l2(nx + 128);
      }
    }

    for (int t = un.t0; t < un.t1; ++t, ++jj) {
      const int b = jj & 1;
      if (!wait_bar(c, BAR_S_FULL + b, (jj >> 1) & 1, LOC_WAIT_S)) return;
      tc_fence_after();
      // every thread observes every completion of O_FULL exactly once and in
      // order (parity waits must never skip a phase): here, for P~V of the
      // previous tile, either before an in-place rescale or at the end of the tile
      bool o_waited = first_tile;
      if (active) {
        if (WINDOW && un.snap && t == un.t0 + 1) {
          // The state after the unit's first key tile goes to a.snap before this tile changes it:
          // P~V of that tile must be complete; the pair adds up its normaliser halves.
          if (!wait_bar(c, BAR_O_FULL, (jj - 1) & 1, LOC_WAIT_O)) return;
          o_waited = true;
          tc_fence_after();
          volatile float* lxs = xch + 2 * (xslot & 1u);
          ++xslot;
          lxs[half] = l_part;
          mbar_arrive(c.bar(BAR_PAIR + quad));
          if (!wait_bar(c, BAR_PAIR + quad, pair_phase & 1, LOC_WAIT_S)) return;
          ++pair_phase;
          const float l_sum = lxs[0] + lxs[1];
          const size_t srow = (size_t)un.h * g.Tp + row;
          float4* dst = reinterpret_cast<float4*>(a.snap.o + srow * D + 64 * half);
          uint32_t rr[64];   // (warp-wide loads; rows past the end of a clipped tile only skip the stores)
          tmem_ld32(tlane + TS_O + 64 * half, *reinterpret_cast<uint32_t(*)[32]>(rr));
          tmem_ld32(tlane + TS_O + 64 * half + 32, *reinterpret_cast<uint32_t(*)[32]>(rr + 32));
          tmem_ld_wait();
          if (row_valid) {
#pragma unroll
            for (int i = 0; i < 8; ++i) st_global_v8(dst + 2 * i, rr + 8 * i);
            if (half == 0) { a.snap.m[srow] = m_ref; a.snap.l[srow] = l_sum; }
          }
        }
        const int tile_lo = tile_key_row<KIND, SPLIT>(un, t);
        const int v_lo = max(un.k0 - tile_lo, 0), v_hi = min(un.k1 - tile_lo, BN);
        const int e_lo = un.x0 - tile_lo, e_hi = un.x1 - tile_lo;
        const bool all_valid = v_lo == 0 && v_hi == BN && (un.x1 <= un.x0 || e_hi <= 0 || e_lo >= BN);
        // the masks of a tile are the same for every row: one bit per column of this thread's half
        // (bit j: column mc + j takes part), built once per tile
        const int mc = HC * half;   // this thread's columns
        auto span_bits = [](int lo, int hi) -> uint64_t {   // bits [lo, hi) of 64
          lo = max(lo, 0);
          hi = min(hi, 64);
          if (hi <= lo) return 0ull;
          return (hi - lo == 64 ? ~0ull : ((1ull << (hi - lo)) - 1ull)) << lo;
        };
        const uint64_t col_bits = all_valid ? ~0ull
                                            : (span_bits(v_lo - mc, v_hi - mc) &
                                               ~((un.x1 > un.x0) ? span_bits(e_lo - mc, e_hi - mc) : 0ull));
        const uint32_t s_addr = tlane + TS_S + 128 * b;
        // This thread's HC scores come out of TMEM once, every load in flight before the one wait (the
        // time of these threads per tile is what bounds a build: a second pass over TMEM and a wait per
        // sixteen columns cost more than the registers).  Columns that take no part are set to -inf here,
        // so that the maximum and the exponentials below need no per-column tests (the common tile has none).
        uint32_t sr[HC];
#pragma unroll
        for (int cb = 0; cb < HC / 16; ++cb)
          tmem_ld16(s_addr + mc + 16 * cb, *reinterpret_cast<uint32_t(*)[16]>(sr + 16 * cb));
        tmem_ld_wait();
        if (!all_valid) {
#pragma unroll
          for (int j = 0; j < HC; ++j) sr[j] = ((col_bits >> j) & 1ull) ? sr[j] : 0xff800000u;
        }
        float mx;
        {
          float m0 = -INFINITY, m1 = -INFINITY, m2 = -INFINITY, m3 = -INFINITY;   // four independent chains
#pragma unroll
          for (int j = 0; j < HC; j += 4) {
            m0 = fmaxf(m0, __uint_as_float(sr[j]));
            m1 = fmaxf(m1, __uint_as_float(sr[j + 1]));
            m2 = fmaxf(m2, __uint_as_float(sr[j + 2]));
            m3 = fmaxf(m3, __uint_as_float(sr[j + 3]));
          }
          mx = fmaxf(fmaxf(m0, m1), fmaxf(m2, m3));
        }
        // The pair's maxima cross through shared memory (the slots alternate between consecutive exchanges).
        // That round trip sits between the maximum and the exponentials of every tile, so a build does not
        // wait for it: after a unit's first tile the reference exponent almost never moves (it moves only
        // when a row's maximum outgrows it by more than RESCALE_SLACK), so the probabilities are formed
        // with the reference as it stands while the exchange is under way, and formed again, the exact
        // way, only when the exchange says that some row of the warp has to move its reference.
        volatile float* mxch = xch + 2 * (xslot & 1u);
        ++xslot;
        mxch[half] = mx;
        mbar_arrive(c.bar(BAR_PAIR + quad));
        float ps0 = 0.f, ps1 = 0.f, ps2 = 0.f, ps3 = 0.f;
        uint32_t pk[HC / 2];
        // Probabilities of this thread's columns, from the registers: P~ = 2^(S c - m) rounded to fp16 (what
        // the P~V product multiplies); the normaliser sums the rounded values, converted back exactly.
        auto probabilities = [&](float m_sub) {
          ps0 = ps1 = ps2 = ps3 = 0.f;
#pragma unroll
          for (int j = 0; j < HC / 2; ++j) {
            const float p0 = ex2(fmaf(__uint_as_float(sr[2 * j]), g.scale_log2, -m_sub));
            const float p1 = ex2(fmaf(__uint_as_float(sr[2 * j + 1]), g.scale_log2, -m_sub));
            const __half2 hp = __floats2half2_rn(p0, p1);
            const float2 pf = __half22float2(hp);
            if (j & 1) { ps2 += pf.x; ps3 += pf.y; } else { ps0 += pf.x; ps1 += pf.y; }
            pk[j] = *reinterpret_cast<const uint32_t*>(&hp);
          }
        };
        // (not for the block queries of a step: few tiles per unit, and that kernel is sensitive to its size;
        // and only after a tile that left every reference of the warp where it was: with large scores the
        // references of a unit's first tiles move often, and forming the probabilities twice costs more
        // than the exchange)
        const bool ahead = !STEP && calm && !__any_sync(0xffffffffu, m_ref == -INFINITY);
        if (ahead) probabilities(m_ref);
        if (!wait_bar(c, BAR_PAIR + quad, pair_phase & 1, LOC_WAIT_S)) return;
        ++pair_phase;
        mx = fmaxf(mxch[0], mxch[1]);
        // integer reference exponent, moved only when the row maximum outgrows it
        // by more than RESCALE_SLACK (so P~ <= 2^RESCALE_SLACK and rescales are rare)
        const float cand = ceilf(mx * g.scale_log2);
        float m_new = m_ref;
        if (m_ref == -INFINITY || cand > m_ref + RESCALE_SLACK) m_new = fmaxf(m_ref, cand);
        float alpha = 1.f;
        // (both warps of the pair see the same rows and the same maxima: they take the same branch)
        calm = !__any_sync(0xffffffffu, m_new != m_ref);
        if (!(ahead && calm)) {
          const float m_use = (m_new == -INFINITY) ? 0.f : m_new;
          if (m_new != m_ref) alpha = (m_ref == -INFINITY) ? 0.f : ex2(m_ref - m_new);
          if ((!first_tile || (WINDOW && have_o)) && __any_sync(0xffffffffu, alpha != 1.f)) {
            // O~ in TMEM is rescaled in place: P~V of the previous tile must be done
            if (!o_waited) {
              if (!wait_bar(c, BAR_O_FULL, (jj - 1) & 1, LOC_WAIT_O)) return;
              o_waited = true;
              tc_fence_after();
            }
#pragma unroll 1
            for (int cb = 0; cb < 4; ++cb) {
              uint32_t rr[16];
              tmem_ld16(tlane + TS_O + 64 * half + 16 * cb, rr);
              tmem_ld_wait();
#pragma unroll
              for (int j = 0; j < 16; ++j) rr[j] = __float_as_uint(__uint_as_float(rr[j]) * alpha);
              tmem_st16(tlane + TS_O + 64 * half + 16 * cb, rr, 0);
            }
          }
          probabilities(m_use);
        }
#pragma unroll
        for (int cb = 0; cb < HC / 16; ++cb)
          tmem_st8(tlane + TS_P + 64 * b + (HC / 2) * half + 8 * cb, *reinterpret_cast<uint32_t(*)[8]>(pk + 8 * cb));
        ps0 += ps2;
        ps1 += ps3;
        const float psum = ps0 + ps1;
        l_part = l_part * alpha + psum;
        m_ref = m_new;
      }
      tmem_st_wait();
      // (before the arrive below: P~V of this tile cannot have been issued yet,
      // so O_FULL is at most one phase ahead of the one waited for)
      if (!o_waited && !wait_bar(c, BAR_O_FULL, (jj - 1) & 1, LOC_WAIT_O)) return;
      tc_fence_before();
      mbar_arrive(c.bar(BAR_P_FULL + b));
      first_tile = false;
    }

    // ---- epilogue ----
    grid_dependency_wait();  // no global store before the preceding grids are complete (see kernel entry)
    // second arrival on Q_FREE (the first is the MMA thread's commit): a 64-row
    // unit stages outside its Q tile, so its Q region may be reloaded at once
    if (un.q_rows != BM && threadIdx.x == 64) mbar_arrive(c.bar(BAR_Q_FREE));
    if (!first_tile) {  // the unit had key tiles: wait for the last P~V
      if (!wait_bar(c, BAR_O_FULL, (jj - 1) & 1, LOC_WAIT_O)) return;
      tc_fence_after();
    }
    // the pair combines its normaliser halves (same alternating slots as the
    // per-tile maximum exchange, which is over for this unit)
    ++epi_unit;
    volatile float* lx = xch + 2 * (xslot & 1u);
    ++xslot;
    lx[half] = l_part;
    if (!epi_sync(c, epi_phase)) return;
    const float l_run = lx[0] + lx[1];
    float mul = (un.epi == EPI_OUT) ? 1.f / l_run : 1.f;
    float mul_rx = 0.f, lse2 = 0.f;   // paired step: weight of the partner's O~, merged log2 normaliser
    if (KIND == KIND_STEP2) {
      const uint32_t rx_row = SM_RX + (uint32_t)r * STAGE_ROW;
      if (un.epi == EPI_SEND) {
        // Second key chunk of its (sequence, head): O~ of the block's rows from TMEM into the partner CTA's
        // receiving buffer (the layout of a staging tile), m and l behind it, then one arrival per thread on
        // the partner's barrier -- the release that makes the stores visible to its acquiring wait.
        const uint32_t peer = cluster_ctarank() ^ 1u;
        const uint32_t dst = mapa_shared(c.base + rx_row, peer);
#pragma unroll 1
        for (int cb = 0; cb < 4; ++cb) {
          uint32_t rr[16];
          if (!first_tile) {
            tmem_ld16(tlane + TS_O + 64 * half + 16 * cb, rr);
            tmem_ld_wait();
          } else {
#pragma unroll
            for (int j = 0; j < 16; ++j) rr[j] = 0u;
          }
          if (row_valid) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const int ch = 16 * half + 4 * cb + i;
              st_cluster_v4(dst + ((ch ^ (r & 7)) << 4), __uint_as_float(rr[4 * i]), __uint_as_float(rr[4 * i + 1]),
                            __uint_as_float(rr[4 * i + 2]), __uint_as_float(rr[4 * i + 3]));
            }
          }
        }
        if (row_valid && half == 0) st_cluster_v2(mapa_shared(c.base + SM_RX_ML + (uint32_t)r * 8u, peer), m_ref, l_run);
        mbar_arrive_cluster(mapa_shared(c.bar(BAR_RX), peer));
        tc_fence_before();
        mbar_arrive(c.bar(BAR_O_FREE));  // (a paired step has one unit per CTA; kept for the barrier's phase count)
        continue;
      }
      // First key chunk: wait (bounded) for the partner's partial state, then merge the two states of the row
      // (Eq. 2-6) into the weights of the two O~ rows; the rows leave through the ordinary output epilogue.
      {
        const uint32_t bar = c.bar(BAR_RX);
        const long long t0 = clock64();
        while (!mbar_try_acquire_cluster(bar, 0u)) {
          if (*c.abort_flag) return;
          if (clock64() - t0 > WAIT_CYCLES) {
            *c.abort_flag = 1;
            if (atomicCAS(c.status, 0, (int)LACACHE_ERR_TIMEOUT) == 0) {
              c.status[1] = LOC_WAIT_O; c.status[2] = blockIdx.x; c.status[3] = threadIdx.x;
            }
            return;
          }
        }
      }
      float m2 = -INFINITY, l2 = 0.f;
      if (row_valid) {
        const float2 ml = *reinterpret_cast<const float2*>(c.gen + SM_RX_ML + r * 8);
        m2 = ml.x; l2 = ml.y;
      }
      const float M = fmaxf(m_ref, m2);
      const float w1 = (m_ref == -INFINITY) ? 0.f : ex2(m_ref - M);
      const float w2 = (m2 == -INFINITY) ? 0.f : ex2(m2 - M);
      const float L = fmaf(l_run, w1, l2 * w2);
      const float inv = 1.f / L;
      mul = w1 * inv;
      mul_rx = w2 * inv;
      lse2 = M + log2f(L);
    }
    if (un.epi == EPI_PARTIAL) {
      // Partial state of this key chunk, straight from TMEM to global memory (each
      // thread 256 contiguous bytes of its row); the last chunk of the (sequence,
      // head) to arrive merges all of them.
      const size_t pbase = ((size_t)un.seq * g.Hq + hrow) * a.max_chunks;  // [chunk][block_len], of this row's head
      const size_t prow0 = (pbase + un.chunk) * g.block_len;
      const int r_blk = unit_row(un, r);
      {
        // (the TMEM loads are warp-wide: rows past the block take part in them and only skip the
        // stores, so a block length that is not a multiple of 32 cannot split a warp around them)
        float4* dst = reinterpret_cast<float4*>(a.part_o + (prow0 + r_blk) * D + 64 * half);
#pragma unroll 1
        for (int cb = 0; cb < 4; ++cb) {
          uint32_t rr[16];
          if (!first_tile) {
            tmem_ld16(tlane + TS_O + 64 * half + 16 * cb, rr);
            tmem_ld_wait();
          } else {
#pragma unroll
            for (int j = 0; j < 16; ++j) rr[j] = 0u;
          }
          if (row_valid) {
#pragma unroll
            for (int i = 0; i < 4; ++i)
              dst[4 * cb + i] = make_float4(__uint_as_float(rr[4 * i]), __uint_as_float(rr[4 * i + 1]),
                                            __uint_as_float(rr[4 * i + 2]), __uint_as_float(rr[4 * i + 3]));
          }
        }
        if (row_valid && half == 0) { a.part_m[prow0 + r_blk] = m_ref; a.part_l[prow0 + r_blk] = l_run; }
      }
      tc_fence_before();
      mbar_arrive(c.bar(BAR_O_FREE));  // the next unit may overwrite O~
      if (!epi_sync(c, epi_phase)) return;  // every partial store of the CTA happens-before thread 64's fence
      if (a.blk_to_state) {  // merged into the rows' state by the launch that follows: nothing to count
        if (un.q_rows == BM && threadIdx.x == 64) mbar_arrive(c.bar(BAR_Q_FREE));
        continue;
      }
      if (threadIdx.x == 64) {
        __threadfence();  // cumulative: publishes the whole CTA's partial state before the counts
        uint32_t last_bits = 0;   // bit j: this chunk was the last of head un.h + j to arrive
        for (int j = 0; j < un.nh; ++j) {
          int* cnt = &a.counters[un.seq * g.Hq + un.h + j];
          const int old = atomicAdd(cnt, 1);
          if (old == un.nchunks - 1) {
            *cnt = 0;
            last_bits |= 1u << j;
          }
        }
        if (last_bits) __threadfence();  // the other chunks' partial states are visible from here on
        *c.flag = last_bits;
      }
      if (!epi_sync(c, epi_phase)) return;
      {
        const uint32_t last_bits = *c.flag;
        for (int j = 0; j < un.nh; ++j)
          if (last_bits & (1u << j))
            merge_partials(g, a, ((size_t)un.seq * g.Hq + un.h + j) * a.max_chunks, un.nchunks, g.block_len, un.row0,
                           un.h + j);
      }
      if (!epi_sync(c, epi_phase)) return;  // the flag may be rewritten
      if (un.q_rows == BM && threadIdx.x == 64) mbar_arrive(c.bar(BAR_Q_FREE));
      continue;
    }
    if (KIND == KIND_BUILD && !SPLIT && un.epi == EPI_STATE && a.st_tma) {
      // Build with one-plane operands: the state of a full row tile goes to a staging tile (four swizzled
      // boxes outside the Q tile and the key / value stages) and leaves as bulk tensor stores issued by the
      // producer thread, so these threads are back at the next unit's tiles after 16 shared-memory stores
      // each instead of eight 32-byte global stores that touch 32 different lines per warp instruction.
      // Every unit takes part in the hand-over (a clipped tile stores the old way and hands over nothing),
      // so the barriers' phases follow the unit count.
      if (uu >= 1 && !wait_bar(c, BAR_ST_FREE, (uu - 1) & 1, LOC_WAIT_O)) return;  // the previous store has read the tile
      if (un.nrows == BM) {
        if (threadIdx.x == 64) mbar_arrive(c.bar(BAR_Q_FREE));
#pragma unroll 1
        for (int cb = 0; cb < 4; ++cb) {     // sixteen features at a time: half a box row
          uint32_t rr[16];
          if (!first_tile) {
            tmem_ld16(tlane + TS_O + 64 * half + 16 * cb, rr);
            tmem_ld_wait();
          } else {
#pragma unroll
            for (int j = 0; j < 16; ++j) rr[j] = 0u;
          }
          uint8_t* const sb = c.gen + st_box(2 * half + (cb >> 1)) + r * 128;
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const int ch = 4 * (cb & 1) + i;
            *reinterpret_cast<float4*>(sb + ((ch ^ (r & 7)) << 4)) =
                make_float4(__uint_as_float(rr[4 * i]), __uint_as_float(rr[4 * i + 1]), __uint_as_float(rr[4 * i + 2]),
                            __uint_as_float(rr[4 * i + 3]));
          }
        }
        if (half == 0) {
          const size_t srow = (size_t)un.h * g.Tp + row;
          a.st.m[srow] = m_ref; a.st.l[srow] = l_run;
        }
        fence_async_smem();   // the bulk stores read the tile through the async proxy
        mbar_arrive(c.bar(BAR_ST_RDY));
        tc_fence_before();
        mbar_arrive(c.bar(BAR_O_FREE));  // the next unit may overwrite O~
        continue;
      }
      mbar_arrive(c.bar(BAR_ST_RDY));   // (nothing staged: the producer answers at once)
    }
    if (un.epi == EPI_STATE && un.q_rows == BM) {
      // Cached state of a build unit, straight from TMEM to global memory (each thread 256
      // contiguous bytes of its row).  Nothing is staged in the Q region, so the next unit's Q
      // tile may be loaded while this epilogue runs.
      if (threadIdx.x == 64) mbar_arrive(c.bar(BAR_Q_FREE));
      const size_t srow = (size_t)un.h * g.Tp + row;
      float4* dst = reinterpret_cast<float4*>(a.st.o + srow * D + 64 * half);
      // (the TMEM loads are warp-wide: rows past the end of a clipped tile take part in them and
      // only skip the stores; first_tile is uniform over the CTA)
      uint32_t rr[64];
      if (!first_tile || (WINDOW && have_o)) {
        tmem_ld32(tlane + TS_O + 64 * half, *reinterpret_cast<uint32_t(*)[32]>(rr));
        tmem_ld32(tlane + TS_O + 64 * half + 32, *reinterpret_cast<uint32_t(*)[32]>(rr + 32));
        tmem_ld_wait();
      } else {
#pragma unroll
        for (int j = 0; j < 64; ++j) rr[j] = 0u;
      }
      if (row_valid) {   // 32-byte stores: whole sectors, half as many instructions
#pragma unroll
        for (int i = 0; i < 8; ++i) st_global_v8(dst + 2 * i, rr + 8 * i);
      }
      if (row_valid && half == 0) { a.st.m[srow] = m_ref; a.st.l[srow] = l_run; }
      if (WINDOW && un.snap && un.t1 - un.t0 <= 1) {
        // a single key tile: the state after it is the final one as well
        float4* sdst = reinterpret_cast<float4*>(a.snap.o + srow * D + 64 * half);
        if (row_valid) {
#pragma unroll
          for (int i = 0; i < 8; ++i) st_global_v8(sdst + 2 * i, rr + 8 * i);
          if (half == 0) { a.snap.m[srow] = m_ref; a.snap.l[srow] = l_run; }
        }
      }
      tc_fence_before();
      mbar_arrive(c.bar(BAR_O_FREE));  // the next unit may overwrite O~
      continue;
    }
    // O~ (this thread's 64 features) from TMEM to its staging row.  The staging
    // area is the Q region (every score MMA of the unit is complete: the last
    // P~V, waited for above, was issued after them); 64-row units use its upper
    // half, which their Q tiles never touch.
    const uint32_t stage_off = SM_Q + (un.q_rows == BM ? 0u : 32768u);
    const bool own_stage = un.q_rows == BM || r < 64;
    uint8_t* const srow = c.gen + stage_off + r * STAGE_ROW;
#pragma unroll 1
    for (int cb = 0; cb < 4; ++cb) {
      uint32_t rr[16];
      if (!first_tile) {
        tmem_ld16(tlane + TS_O + 64 * half + 16 * cb, rr);
        tmem_ld_wait();
      } else {
#pragma unroll
        for (int j = 0; j < 16; ++j) rr[j] = 0u;
      }
      if (own_stage) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int ch = 16 * half + 4 * cb + i;
          float4 v = make_float4(__uint_as_float(rr[4 * i]) * mul, __uint_as_float(rr[4 * i + 1]) * mul,
                                 __uint_as_float(rr[4 * i + 2]) * mul, __uint_as_float(rr[4 * i + 3]) * mul);
          if (KIND == KIND_STEP2 && row_valid) {   // + the partner chunk's O~, weighted
            const float4 p = *reinterpret_cast<const float4*>(c.gen + SM_RX + r * STAGE_ROW + ((ch ^ (r & 7)) << 4));
            v.x = fmaf(p.x, mul_rx, v.x); v.y = fmaf(p.y, mul_rx, v.y);
            v.z = fmaf(p.z, mul_rx, v.z); v.w = fmaf(p.w, mul_rx, v.w);
          }
          *reinterpret_cast<float4*>(srow + ((ch ^ (r & 7)) << 4)) = v;
        }
      }
    }
    tc_fence_before();
    mbar_arrive(c.bar(BAR_O_FREE));  // the next unit may overwrite O~
    if (un.epi == EPI_STATE) {
      const size_t srow = (size_t)un.h * g.Tp + row;
      if (row_valid && half == 0) { a.st.m[srow] = m_ref; a.st.l[srow] = l_run; }
      if (!epi_sync(c, epi_phase)) return;
      coop_store_rows(c, stage_off, a.st.o + ((size_t)un.h * g.Tp + un.row0) * D, D, un.nrows);
    } else if (un.epi == EPI_OUT) {
      const size_t orow = (size_t)row * g.Hq + hrow;
      if (row_valid && half == 0 && a.lse) a.lse[orow] = (KIND == KIND_STEP2 ? lse2 : m_ref + log2f(l_run)) * LN2;
      if (!epi_sync(c, epi_phase)) return;
      for (int j = 0; j < un.nh; ++j)   // one head's rows at a time (a single head unless block queries are packed)
        coop_store_out_rows(c, a, stage_off + (uint32_t)(j * un.rh) * STAGE_ROW, ((size_t)un.row0 * g.Hq + un.h + j) * D,
                            (size_t)g.Hq * D, un.nrows);
    }
    if (!epi_sync(c, epi_phase)) return;  // the staging rows have been read
    if (un.q_rows == BM && threadIdx.x == 64) mbar_arrive(c.bar(BAR_Q_FREE));  // the Q region may be reloaded
  }
}

// Output rows [row0, row0 + nrows) of head h from a swizzled staging tile (four boxes of
// 32 features x 128 rows) to the caller's `out` with tiled bulk stores: one 128-row box, or
// for a clipped tile boxes of 64, 32, 16 and 8 rows (each starts on a multiple of 8 rows,
// where the staging tile's swizzle pattern repeats).  Returns the rows covered; the last
// nrows % 8 rows are left to the row threads.  The caller commits the bulk group.
// With a bf16 `out` the tile holds two boxes of 64 bf16 features x 128 rows, at the places of the fp32
// boxes 0 and 2, and the tensor maps describe bf16 boxes.
__device__ __forceinline__ int store_out_tile(const TcMaps& maps, uint32_t src, int h, int row0, int nrows,
                                              bool bf16) {
  const int nb = bf16 ? 2 : 4;                     // boxes per tile
  const uint32_t bstep = bf16 ? 2 * IO_BOX : IO_BOX;
  const int fstep = bf16 ? 64 : 32;                // features per box
  if (nrows == BM) {
    for (int cb = 0; cb < nb; ++cb) tma_store_3d(&maps.out, src + cb * bstep, fstep * cb, h, row0);
    return BM;
  }
  int done = 0;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int bs = 64 >> i;
    if (nrows - done >= bs) {
      for (int cb = 0; cb < nb; ++cb)
        tma_store_3d(&maps.out_sub[i], src + cb * bstep + done * 128, fstep * cb, h, row0 + done);
      done += bs;
    }
  }
  return done;
}

// The merge roles' combine, out = (alpha O~_cache + P~V) / l, for this thread's 64 features of tile row r, in
// place in the staging tile: `sbox` is the row's place in the thread's first fp32 box (box 2 * half; the
// second follows IO_BOX further), `o_tmem` the TMEM address of its 64 P~V columns.  With a bf16 `out` the 64
// results are packed and written over the row of the first box (128 bytes, the layout of a bf16 box).
__device__ __forceinline__ void combine_row(uint8_t* sbox, int sw, uint32_t o_tmem, float a_inv, float inv, bool bf16) {
  if (!bf16) {
#pragma unroll
    for (int q2 = 0; q2 < 2; ++q2) {
      uint32_t rr[32];
      tmem_ld32(o_tmem + 32 * q2, rr);
      tmem_ld_wait();
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        float4* p4 = reinterpret_cast<float4*>(sbox + q2 * IO_BOX + ((i ^ sw) << 4));
        float4 oc = *p4;
        oc.x = fmaf(oc.x, a_inv, __uint_as_float(rr[4 * i]) * inv);
        oc.y = fmaf(oc.y, a_inv, __uint_as_float(rr[4 * i + 1]) * inv);
        oc.z = fmaf(oc.z, a_inv, __uint_as_float(rr[4 * i + 2]) * inv);
        oc.w = fmaf(oc.w, a_inv, __uint_as_float(rr[4 * i + 3]) * inv);
        *p4 = oc;
      }
    }
    return;
  }
  uint32_t pk[32];   // 64 bf16 results
#pragma unroll
  for (int q2 = 0; q2 < 2; ++q2) {
    uint32_t rr[32];
    tmem_ld32(o_tmem + 32 * q2, rr);
    tmem_ld_wait();
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float4 oc = *reinterpret_cast<const float4*>(sbox + q2 * IO_BOX + ((i ^ sw) << 4));
      pk[16 * q2 + 2 * i] = pack_bf16x2(fmaf(oc.x, a_inv, __uint_as_float(rr[4 * i]) * inv),
                                        fmaf(oc.y, a_inv, __uint_as_float(rr[4 * i + 1]) * inv));
      pk[16 * q2 + 2 * i + 1] = pack_bf16x2(fmaf(oc.z, a_inv, __uint_as_float(rr[4 * i + 2]) * inv),
                                            fmaf(oc.w, a_inv, __uint_as_float(rr[4 * i + 3]) * inv));
    }
  }
  // (every read of the row's two fp32 boxes is done: only this thread touches them)
#pragma unroll
  for (int j = 0; j < 8; ++j)
    *reinterpret_cast<uint4*>(sbox + ((j ^ sw) << 4)) = make_uint4(pk[4 * j], pk[4 * j + 1], pk[4 * j + 2], pk[4 * j + 3]);
}
// one row of a clipped tile's tail, from the staging tile straight to `out` (this thread's 64 features)
__device__ __forceinline__ void store_tail_row(const AttnArgs& a, const uint8_t* sbox, int sw, size_t orow, int half) {
  if (a.out_bf16) {
    uint4* dst = reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(a.out) + orow * D + 64 * half);
#pragma unroll
    for (int j = 0; j < 8; ++j) dst[j] = *reinterpret_cast<const uint4*>(sbox + ((j ^ sw) << 4));
  } else {
    float4* dst = reinterpret_cast<float4*>(a.out + orow * D + 64 * half);
#pragma unroll
    for (int q2 = 0; q2 < 2; ++q2)
#pragma unroll
      for (int i = 0; i < 8; ++i)
        dst[8 * q2 + i] = *reinterpret_cast<const float4*>(sbox + q2 * IO_BOX + ((i ^ sw) << 4));
  }
}

// ===========================================================================
// merge role: fixed queries x block keys, merged into the cached state
// ===========================================================================
template <bool SPLIT>
__device__ void merge_producer(const Cta& c, const TcMaps& maps, const Geometry& g, const AttnArgs& a, int first,
                               int stride, int n_units, WorkItem it) {
  int uu = 0;
  for (int u = first; u < n_units; u += stride, ++uu) {
    WorkItem nxt = it;
    if (u + stride < n_units) nxt = load_item(a.items_merge + (u + stride) / g.Hq);
    const int h = u % g.Hq;
    const int b = uu & 1, k = uu >> 1;
    if (uu >= 1 && !wait_bar(c, BAR_Q_FREE, (uu - 1) & 1, LOC_WAIT_Q)) return;
    load_q_tile<SPLIT>(c, maps, BM, it.row0, h);
    if (uu == 0) {
      // first unit: the cached O~ tile does not depend on the RoPE kernel launched
      // just before this one, the block's keys and values do: wait for that grid
      // only now (this kernel may have started early)
      mbar_expect_tx(c.bar(BAR_IO_FULL), 4 * IO_BOX);
#pragma unroll
      for (int cb = 0; cb < 4; ++cb)
        tma_load_3d(c.base + SM_IO + cb * IO_BOX, &maps.st_o, c.bar(BAR_IO_FULL), 32 * cb, it.row0, h);
      grid_dependency_wait();
      load_kv_tile<SPLIT>(maps, c.base + SM_KV, c.bar(BAR_KV_FULL), it.blk_start, h / g.group);
    } else {
      // later units: keys first (their stage frees early), then the cached O~
      // tile (four boxes of 32 features x 128 rows; rows past nrows are read but
      // never used) once the previous unit's output has left the staging tile
      if (k >= 1 && !wait_bar(c, BAR_KV_FREE + b, (k - 1) & 1, LOC_WAIT_K)) return;
      load_kv_tile<SPLIT>(maps, c.base + SM_KV + b * KV_STAGE, c.bar(BAR_KV_FULL + b), it.blk_start, h / g.group);
      if (!wait_bar(c, BAR_IO_FREE, (uu - 1) & 1, LOC_WAIT_V)) return;
      mbar_expect_tx(c.bar(BAR_IO_FULL), 4 * IO_BOX);
#pragma unroll
      for (int cb = 0; cb < 4; ++cb)
        tma_load_3d(c.base + SM_IO + cb * IO_BOX, &maps.st_o, c.bar(BAR_IO_FULL), 32 * cb, it.row0, h);
    }
    it = nxt;
  }
}

template <bool SPLIT>
__device__ void merge_mma(const Cta& c, const Geometry& g, const AttnArgs& a, int first, int stride, int n_units) {
  const int n_s = (g.block_len + 15) & ~15;  // score columns (keys), a multiple of 16
  const uint32_t idesc_s = idesc_f16((!SPLIT && g.op_f16) ? 0u : 1u, 0u, BM, (uint32_t)n_s);
  int uu = 0;
  if (first < n_units) {
    if (!wait_bar(c, BAR_Q_FULL, 0, LOC_WAIT_Q)) return;
    if (!wait_bar(c, BAR_KV_FULL, 0, LOC_WAIT_K)) return;
    tc_fence_after();
    issue_s_mma<SPLIT>(c.base + SM_Q, BM * 128u, c.base + SM_KV, c.base + SM_KV + KV_KLO, K_BOX, c.tmem + TM_S, idesc_s);
    tc_commit(c.bar(BAR_S_FULL));
    tc_commit(c.bar(BAR_Q_FREE));
  }
  for (int u = first; u < n_units; u += stride, ++uu) {
    const int b = uu & 1, k = uu >> 1;
    if (!wait_bar(c, BAR_P_FULL + b, k & 1, LOC_WAIT_S)) return;
    if (k >= 1 && !wait_bar(c, BAR_O_FREE + b, (k - 1) & 1, LOC_WAIT_O)) return;
    tc_fence_after();
    issue_pv_mma(c.base + SM_KV + b * KV_STAGE + KV_V, K_BOX, c.tmem + TM_P + 32 * b, c.tmem + TM_O + 128 * b, n_s / 16,
                 0u);
    tc_commit(c.bar(BAR_O_FULL + b));
    tc_commit(c.bar(BAR_KV_FREE + b));
    if (u + stride < n_units) {  // scores of the next unit as soon as its tiles land
      const int bn = (uu + 1) & 1;
      if (!wait_bar(c, BAR_Q_FULL, (uu + 1) & 1, LOC_WAIT_Q)) return;
      if (!wait_bar(c, BAR_KV_FULL + bn, ((uu + 1) >> 1) & 1, LOC_WAIT_K)) return;
      tc_fence_after();
      issue_s_mma<SPLIT>(c.base + SM_Q, BM * 128u, c.base + SM_KV + bn * KV_STAGE, c.base + SM_KV + bn * KV_STAGE + KV_KLO, K_BOX,
                  c.tmem + TM_S + 64 * bn, idesc_s);
      tc_commit(c.bar(BAR_S_FULL + bn));
      tc_commit(c.bar(BAR_Q_FREE));
    }
  }
}

__device__ void merge_rows(const Cta& c, const TcMaps& maps, const Geometry& g, const AttnArgs& a, int first,
                           int stride, int n_units, WorkItem it) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int quad = warp & 3;
  const int half = (warp - 2) >> 2;
  const int r = quad * 32 + lane;
  const uint32_t tlane = c.tmem + ((uint32_t)(quad * 32) << 16);
  const float LN2 = 0.69314718055994530942f;
  const int n_s = (g.block_len + 15) & ~15;
  const int L = g.block_len;
  // staging layout (as TMA writes and reads it): box cb = features [32 cb, 32 cb + 32),
  // row r at +128 r, its 16-byte chunk j at ((j ^ (r & 7)) << 4)
  uint8_t* const sbox = c.gen + SM_IO + (2 * half) * IO_BOX + r * 128;
  const int sw = r & 7;
  uint32_t epi_phase = 0;
  int uu = 0;
  for (int u = first; u < n_units; u += stride, ++uu) {
    WorkItem nxt = it;
    if (u + stride < n_units) nxt = load_item(a.items_merge + (u + stride) / g.Hq);
    const int h = u % g.Hq;
    const int b = uu & 1, par = (uu >> 1) & 1;
    const int row = it.row0 + r;
    const bool row_valid = r < it.nrows;
    const size_t srow = (size_t)h * g.Tp + row;
    float m_c = -INFINITY, l_c = 0.f;
    if (row_valid) { m_c = __ldg(a.st.m + srow); l_c = __ldg(a.st.l + srow); }

    if (!wait_bar(c, BAR_S_FULL + b, par, LOC_WAIT_S)) return;
    tc_fence_after();
    // scores against the block's keys: columns [0, block_len) are valid
    float mx = -INFINITY;
    uint32_t s0[32], s1[32];
    tmem_ld32(tlane + TM_S + 64 * b, s0);
    if (n_s > 32) tmem_ld32(tlane + TM_S + 64 * b + 32, s1);
    tmem_ld_wait();
#pragma unroll
    for (int j = 0; j < 32; ++j)
      if (j < L) mx = fmaxf(mx, __uint_as_float(s0[j]));
    if (n_s > 32) {
#pragma unroll
      for (int j = 0; j < 32; ++j)
        if (32 + j < L) mx = fmaxf(mx, __uint_as_float(s1[j]));
    }
    const float m_new = fmaxf(m_c, ceilf(mx * g.scale_log2));
    const float alpha = (m_c == -INFINITY) ? 0.f : ex2(m_c - m_new);
    float psum = 0.f;
    {
      uint32_t pk[16];
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        float p0 = (2 * j < L) ? round_to_half_bits(ex2(fmaf(__uint_as_float(s0[2 * j]), g.scale_log2, -m_new))) : 0.f;
        float p1 = (2 * j + 1 < L) ? round_to_half_bits(ex2(fmaf(__uint_as_float(s0[2 * j + 1]), g.scale_log2, -m_new))) : 0.f;
        psum += p0 + p1;
        __half2 hp = __floats2half2_rn(p0, p1);
        pk[j] = *reinterpret_cast<uint32_t*>(&hp);
      }
      if (half == 0) tmem_st16(tlane + TM_P + 32 * b, pk);
      if (n_s > 32) {
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          float p0 = (32 + 2 * j < L) ? round_to_half_bits(ex2(fmaf(__uint_as_float(s1[2 * j]), g.scale_log2, -m_new))) : 0.f;
          float p1 = (33 + 2 * j < L) ? round_to_half_bits(ex2(fmaf(__uint_as_float(s1[2 * j + 1]), g.scale_log2, -m_new))) : 0.f;
          psum += p0 + p1;
          __half2 hp = __floats2half2_rn(p0, p1);
          pk[j] = *reinterpret_cast<uint32_t*>(&hp);
        }
        if (half == 1) tmem_st16(tlane + TM_P + 32 * b + 16, pk);
      }
    }
    tmem_st_wait();
    tc_fence_before();
    mbar_arrive(c.bar(BAR_P_FULL + b));
    const float l_new = fmaf(l_c, alpha, psum);
    const float inv = 1.f / l_new;
    const float a_inv = alpha * inv;

    if (!wait_bar(c, BAR_O_FULL + b, par, LOC_WAIT_O)) return;
    if (!wait_bar(c, BAR_IO_FULL, uu & 1, LOC_WAIT_V)) return;
    tc_fence_after();
    // out = (alpha O~_cache + P~V) / l, in place in the staging tile
    combine_row(sbox, sw, tlane + TM_O + 128 * b + 64 * half, a_inv, inv, a.out_bf16 != 0);
    tc_fence_before();
    mbar_arrive(c.bar(BAR_O_FREE + b));
    grid_dependency_wait();  // no global store before the preceding grids are complete
    const size_t orow = (size_t)row * g.Hq + h;
    if (row_valid && half == 0 && a.lse) a.lse[orow] = (m_new + log2f(l_new)) * LN2;
    if (row_valid && r >= (it.nrows & ~7)) {
      // the last nrows % 8 rows of a clipped tile go out one by one (the rest by bulk stores)
      store_tail_row(a, sbox, sw, orow, half);
    }
    fence_async_smem();
    if (!epi_sync(c, epi_phase)) return;  // the whole tile is in the staging buffer
    if (threadIdx.x == 64) {
      grid_dependency_wait();
      if (store_out_tile(maps, c.base + SM_IO, h, it.row0, it.nrows, a.out_bf16 != 0) > 0) {
        bulk_commit();
        bulk_wait_read();               // the copies have read the staging tile
      }
      mbar_arrive(c.bar(BAR_IO_FREE));  // the producer may load the next tile
    }
    it = nxt;
  }
}

// ===========================================================================
// ===========================================================================
// merge role, pipelined variant for block_len <= 32.  The block's keys and
// values need only 24 KB, which leaves room for two staging tiles of cached
// O~: the tile of unit u + 1 streams in while unit u is combined and while the
// output of unit u - 1 streams out, so a CTA keeps ~190 KB of loads and stores
// in flight instead of one tile at a time.  Keys and values have separate
// barriers (single stage each: the next unit's keys load as soon as the
// current scores are done).  The producer thread also issues the output
// stores, and every role reads the CTA's units from a table in shared memory.
// ===========================================================================
constexpr uint32_t DM_IO = 65536;                      // two staging tiles of 4 boxes (64 KB each)
constexpr uint32_t DM_IO_TILE = 4 * IO_BOX;
constexpr uint32_t DM_KBOX = 32 * 128;                 // one [32 rows][64 cols] 16-bit box
constexpr uint32_t DM_K = DM_IO + 2 * DM_IO_TILE;      // K hi (2 boxes), K lo (2 boxes)
constexpr uint32_t DM_V = DM_K + 4 * DM_KBOX;          // V (2 boxes)
constexpr uint32_t DM_TAB = DM_V + 2 * DM_KBOX;        // unit table: {row0, nrows, blk_start, head}
constexpr int DM_MAX_UNITS = (int)((SM_XCH - DM_TAB) / 16);
static_assert(DM_TAB % 16 == 0 && DM_MAX_UNITS >= TC_DEEP_MAX_UNITS, "unit table");

struct DUnit { int row0, nrows, blk_start, h, seq; };
__device__ __forceinline__ DUnit deep_unit(const Cta& c, int i) {
  const int4 v = *reinterpret_cast<const int4*>(c.gen + DM_TAB + 16 * i);
  return DUnit{v.x, v.y, v.z, v.w & 0xFFFF, v.w >> 16};
}

template <bool SPLIT>
__device__ void deep_producer(const Cta& c, const TcMaps& maps, const Geometry& g, int n_my, bool kv_computed,
                              bool out_bf16) {
  if (n_my == 0) return;
  auto load_q = [&](int i) {
    const DUnit un = deep_unit(c, i);
    load_q_tile<SPLIT>(c, maps, BM, un.row0, un.h);
  };
  auto load_io = [&](int i) {
    const DUnit un = deep_unit(c, i);
    const uint32_t bar = c.bar((i & 1) ? BAR_IO_FULL1 : BAR_IO_FULL);
    const uint32_t dst = c.base + DM_IO + (i & 1) * DM_IO_TILE;
    mbar_expect_tx(bar, DM_IO_TILE);
#pragma unroll
    for (int cb = 0; cb < 4; ++cb) tma_load_3d(dst + cb * IO_BOX, &maps.st_o, bar, 32 * cb, un.row0, un.h);
  };
  auto load_k = [&](int i) {
    const DUnit un = deep_unit(c, i);
    const uint32_t bar = c.bar(BAR_KV_FULL), kb = c.base + DM_K;
    const int kh = un.h / g.group;
    mbar_expect_tx(bar, (SPLIT ? 4 : 2) * DM_KBOX);
    load_qk_box(kb, &maps.k32, bar, un.blk_start, kh);
  };
  auto load_v = [&](int i) {
    const DUnit un = deep_unit(c, i);
    const uint32_t bar = c.bar(BAR_KV_FULL1), vb = c.base + DM_V;
    const int kh = un.h / g.group;
    mbar_expect_tx(bar, 2 * DM_KBOX);
    load_v_box(vb, &maps.v32, bar, un.blk_start, kh);
  };
  // Q' and cached O~ of fixed rows do not depend on the RoPE kernel launched
  // just before this one; the block's keys and values do
  // (the second unit's cached-O~ tile is requested once the first Q' tile has landed, not with it: at the start
  // of a step every CTA's requests queue in front of HBM, and the tile that is needed last gives way)
  load_q(0);
  load_io(0);
  bool dep_done = false;
  bool q0_landed = false;   // (latched: the barrier's parity comes round again)
  if (kv_computed) {
    // the row threads rotate / convert the block's keys and values of the first unit
    // from the raw inputs (plain arrivals keep the barriers' phase counts in step)
    mbar_arrive(c.bar(BAR_KV_FULL));
    mbar_arrive(c.bar(BAR_KV_FULL1));
  } else {
    grid_dependency_wait();
    dep_done = true;
    load_k(0);
    load_v(0);
  }
  int qu = 1, ku = 1, vu = 1, iu = 1, su = 0;
  bool pending_read = false;  // an output store may still be reading its staging tile
  long long t_idle = 0;
  while (su < n_my) {
    bool did = false;
    if (qu < n_my && mbar_test(c.bar(BAR_Q_FREE), (qu - 1) & 1)) { load_q(qu); ++qu; did = true; }
    if (ku < n_my && mbar_test(c.bar(BAR_KV_FREE), (ku - 1) & 1)) {
      if (!dep_done) { grid_dependency_wait(); dep_done = true; }  // long over by now
      load_k(ku); ++ku; did = true;
    }
    if (vu < n_my && mbar_test(c.bar(BAR_KV_FREE1), (vu - 1) & 1)) {
      if (!dep_done) { grid_dependency_wait(); dep_done = true; }
      load_v(vu); ++vu; did = true;
    }
    if (mbar_test(c.bar((su & 1) ? BAR_OUT_RDY1 : BAR_OUT_RDY), (su >> 1) & 1)) {
      const DUnit un = deep_unit(c, su);
      if (!dep_done) { grid_dependency_wait(); dep_done = true; }  // no store before the preceding grids are complete
      if (store_out_tile(maps, c.base + DM_IO + (su & 1) * DM_IO_TILE, un.h, un.row0, un.nrows, out_bf16) > 0) {
        bulk_commit();
        pending_read = true;
      }
      ++su;
      did = true;
    }
    if (!q0_landed && mbar_test(c.bar(BAR_Q_FULL), 0)) q0_landed = true;
    if (!did && iu < n_my && su > iu - 2 && q0_landed) {  // the tile of unit iu - 2 has been handed to its store
      if (pending_read) { bulk_wait_read(); pending_read = false; }
      load_io(iu);
      ++iu;
      did = true;
    }
    if (did) {
      t_idle = 0;
    } else {
      if (t_idle == 0) t_idle = clock64();
      if (*c.abort_flag) break;
      if (clock64() - t_idle > WAIT_CYCLES) {
        *c.abort_flag = 1;
        if (atomicCAS(c.status, 0, (int)LACACHE_ERR_TIMEOUT) == 0) {
          c.status[1] = LOC_WAIT_V; c.status[2] = blockIdx.x; c.status[3] = threadIdx.x;
        }
        break;
      }
    }
  }
  bulk_wait_read();  // shared memory stays valid until the last store has read it
}

template <bool SPLIT>
__device__ void deep_mma(const Cta& c, const Geometry& g, int n_my, bool kv_computed) {
  if (n_my == 0) return;
  const int n_s = (g.block_len + 15) & ~15;
  const uint32_t idesc_s = idesc_f16((!SPLIT && g.op_f16) ? 0u : 1u, 0u, BM, (uint32_t)n_s);
  const uint32_t kb = c.base + DM_K;
  if (!wait_bar(c, BAR_Q_FULL, 0, LOC_WAIT_Q)) return;
  if (!wait_bar(c, BAR_KV_FULL, 0, LOC_WAIT_K)) return;
  if (kv_computed && !wait_bar(c, BAR_QC, 0, LOC_WAIT_K)) return;  // keys and values written by the row threads
  tc_fence_after();
  issue_s_mma<SPLIT>(c.base + SM_Q, BM * 128u, kb, kb + 2 * DM_KBOX, DM_KBOX, c.tmem + TM_S, idesc_s);
  tc_commit(c.bar(BAR_S_FULL));
  tc_commit(c.bar(BAR_Q_FREE));
  tc_commit(c.bar(BAR_KV_FREE));
  for (int uu = 0; uu < n_my; ++uu) {
    const int b = uu & 1, k = uu >> 1;
    if (!wait_bar(c, BAR_P_FULL + b, k & 1, LOC_WAIT_S)) return;
    if (k >= 1 && !wait_bar(c, BAR_O_FREE + b, (k - 1) & 1, LOC_WAIT_O)) return;
    if (!wait_bar(c, BAR_KV_FULL1, uu & 1, LOC_WAIT_V)) return;
    tc_fence_after();
    issue_pv_mma(c.base + DM_V, DM_KBOX, c.tmem + TM_P + 32 * b, c.tmem + TM_O + 128 * b, n_s / 16, 0u);
    tc_commit(c.bar(BAR_O_FULL + b));
    tc_commit(c.bar(BAR_KV_FREE1));
    if (uu + 1 < n_my) {  // scores of the next unit as soon as its tiles land
      const int bn = (uu + 1) & 1;
      if (!wait_bar(c, BAR_Q_FULL, (uu + 1) & 1, LOC_WAIT_Q)) return;
      if (!wait_bar(c, BAR_KV_FULL, (uu + 1) & 1, LOC_WAIT_K)) return;
      tc_fence_after();
      issue_s_mma<SPLIT>(c.base + SM_Q, BM * 128u, kb, kb + 2 * DM_KBOX, DM_KBOX, c.tmem + TM_S + 64 * bn, idesc_s);
      tc_commit(c.bar(BAR_S_FULL + bn));
      tc_commit(c.bar(BAR_Q_FREE));
      tc_commit(c.bar(BAR_KV_FREE));
    }
  }
}

template <bool SPLIT>
__device__ void deep_rows(const Cta& c, const Geometry& g, const AttnArgs& a, int n_my) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int quad = warp & 3;
  const int half = (warp - 2) >> 2;
  const int r = quad * 32 + lane;
  const uint32_t tlane = c.tmem + ((uint32_t)(quad * 32) << 16);
  const float LN2 = 0.69314718055994530942f;
  const int L = g.block_len;
  const int sw = r & 7;
  // the cached (m, l) of a unit's rows are fetched one unit ahead
  float m_nx = -INFINITY, l_nx = 0.f;
  if (n_my > 0) {
    const DUnit un = deep_unit(c, 0);
    if (r < un.nrows) {
      const size_t srow = (size_t)un.h * g.Tp + un.row0 + r;
      m_nx = __ldg(a.st.m + srow);
      l_nx = __ldg(a.st.l + srow);
    }
  }
  if (n_my > 0 && a.k_raw != nullptr) {
    // First unit: the block's keys (rotated, split bf16) and values (fp16) of this head,
    // computed here with the RoPE kernel's own arithmetic and written where the TMA loads
    // would have put them ([plane][feature half][row][64], 16-byte chunks XOR-swizzled by
    // the row), so the unit does not wait for that kernel.
    const DUnit un = deep_unit(c, 0);
    const int kh = un.h / g.group;
    const int tq = threadIdx.x - 64;
    for (int i = tq; i < L * 8; i += ROW_THREADS) {
      const int ki = i >> 3, ch = i & 7, c0 = ch * 8;
      const size_t src = (size_t)un.seq * L + ki;
      const size_t soff = (src * g.Hkv + kh) * D;
      float x1[8], x2[8], cs[8], sn[8], y1[8], y2[8];
      rope_load8(a.k_raw, soff + c0, true, x1);
      rope_load8(a.k_raw, soff + c0 + D / 2, true, x2);
      const float4* cp = reinterpret_cast<const float4*>(a.row_cos + src * (D / 2) + c0);
      const float4* sp = reinterpret_cast<const float4*>(a.row_sin + src * (D / 2) + c0);
      const float4 ca = cp[0], cb = cp[1], sa = sp[0], sb = sp[1];
      cs[0] = ca.x; cs[1] = ca.y; cs[2] = ca.z; cs[3] = ca.w; cs[4] = cb.x; cs[5] = cb.y; cs[6] = cb.z; cs[7] = cb.w;
      sn[0] = sa.x; sn[1] = sa.y; sn[2] = sa.z; sn[3] = sa.w; sn[4] = sb.x; sn[5] = sb.y; sn[6] = sb.z; sn[7] = sb.w;
      rope_rotate8(x1, x2, cs, sn, y1, y2);
      uint4 h1, l1, h2, l2;
      if (!SPLIT && g.op_f16) {
        h1 = rope_half8(y1);
        h2 = rope_half8(y2);
      } else {
        rope_split8(y1, h1, l1);
        rope_split8(y2, h2, l2);
      }
      uint8_t* const k0 = c.gen + DM_K + ki * 128 + ((ch ^ (ki & 7)) << 4);
      *reinterpret_cast<uint4*>(k0) = h1;
      *reinterpret_cast<uint4*>(k0 + DM_KBOX) = h2;
      if (SPLIT) {
        *reinterpret_cast<uint4*>(k0 + 2 * DM_KBOX) = l1;
        *reinterpret_cast<uint4*>(k0 + 3 * DM_KBOX) = l2;
      }
      // values: the same two 8-feature chunks of row ki, unrotated
      float v1[8], v2[8];
      rope_load8(a.v_raw, soff + c0, true, v1);
      rope_load8(a.v_raw, soff + c0 + D / 2, true, v2);
      uint8_t* const v0 = c.gen + DM_V + ki * 128 + ((ch ^ (ki & 7)) << 4);
      *reinterpret_cast<uint4*>(v0) = rope_half8(v1);
      *reinterpret_cast<uint4*>(v0 + DM_KBOX) = rope_half8(v2);
    }
    // rows [L, 32) of the boxes (block_len < 32) are never multiplied by a non-zero P~
    // but must not hold NaN or Inf patterns: clear them
    for (int i = tq + L * 8; i < 32 * 8; i += ROW_THREADS) {
      const int ki = i >> 3, ch = i & 7;
      const uint4 z = make_uint4(0u, 0u, 0u, 0u);
      uint8_t* const k0 = c.gen + DM_K + ki * 128 + ((ch ^ (ki & 7)) << 4);
      *reinterpret_cast<uint4*>(k0) = z; *reinterpret_cast<uint4*>(k0 + DM_KBOX) = z;
      if (SPLIT) { *reinterpret_cast<uint4*>(k0 + 2 * DM_KBOX) = z; *reinterpret_cast<uint4*>(k0 + 3 * DM_KBOX) = z; }
      uint8_t* const v0 = c.gen + DM_V + ki * 128 + ((ch ^ (ki & 7)) << 4);
      *reinterpret_cast<uint4*>(v0) = z; *reinterpret_cast<uint4*>(v0 + DM_KBOX) = z;
    }
    fence_async_smem();  // the MMAs read shared memory through the async proxy
    mbar_arrive(c.bar(BAR_QC));
  }
  for (int uu = 0; uu < n_my; ++uu) {
    const DUnit un = deep_unit(c, uu);
    const int b = uu & 1, par = (uu >> 1) & 1;
    const int row = un.row0 + r;
    const bool row_valid = r < un.nrows;
    const float m_c = m_nx, l_c = l_nx;
    m_nx = -INFINITY; l_nx = 0.f;
    if (uu + 1 < n_my) {
      const DUnit nx = deep_unit(c, uu + 1);
      if (r < nx.nrows) {
        const size_t srow = (size_t)nx.h * g.Tp + nx.row0 + r;
        m_nx = __ldg(a.st.m + srow);
        l_nx = __ldg(a.st.l + srow);
      }
    }
    // staging tile b (as TMA writes and reads it): box cb = features [32 cb, 32 cb + 32),
    // row r at +128 r, its 16-byte chunk j at ((j ^ (r & 7)) << 4)
    uint8_t* const sbox = c.gen + DM_IO + b * DM_IO_TILE + (2 * half) * IO_BOX + r * 128;

    if (!wait_bar(c, BAR_S_FULL + b, par, LOC_WAIT_S)) return;
    tc_fence_after();
    float mx = -INFINITY;
    uint32_t s0[32];
    tmem_ld32(tlane + TM_S + 64 * b, s0);
    tmem_ld_wait();
#pragma unroll
    for (int j = 0; j < 32; ++j)
      if (j < L) mx = fmaxf(mx, __uint_as_float(s0[j]));
    const float m_new = fmaxf(m_c, ceilf(mx * g.scale_log2));
    const float alpha = (m_c == -INFINITY) ? 0.f : ex2(m_c - m_new);
    float psum = 0.f;
    {
      uint32_t pk[16];
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        float p0 = (2 * j < L) ? round_to_half_bits(ex2(fmaf(__uint_as_float(s0[2 * j]), g.scale_log2, -m_new))) : 0.f;
        float p1 = (2 * j + 1 < L) ? round_to_half_bits(ex2(fmaf(__uint_as_float(s0[2 * j + 1]), g.scale_log2, -m_new))) : 0.f;
        psum += p0 + p1;
        __half2 hp = __floats2half2_rn(p0, p1);
        pk[j] = *reinterpret_cast<uint32_t*>(&hp);
      }
      if (half == 0) tmem_st16(tlane + TM_P + 32 * b, pk);
    }
    tmem_st_wait();
    tc_fence_before();
    mbar_arrive(c.bar(BAR_P_FULL + b));
    const float l_new = fmaf(l_c, alpha, psum);
    const float inv = 1.f / l_new;
    const float a_inv = alpha * inv;

    if (!wait_bar(c, BAR_O_FULL + b, par, LOC_WAIT_O)) return;
    if (!wait_bar(c, b ? BAR_IO_FULL1 : BAR_IO_FULL, par, LOC_WAIT_V)) return;
    tc_fence_after();
    // out = (alpha O~_cache + P~V) / l, in place in the staging tile
    combine_row(sbox, sw, tlane + TM_O + 128 * b + 64 * half, a_inv, inv, a.out_bf16 != 0);
    tc_fence_before();
    mbar_arrive(c.bar(BAR_O_FREE + b));
    grid_dependency_wait();  // no global store before the preceding grids are complete
    const size_t orow = (size_t)row * g.Hq + un.h;
    if (row_valid && half == 0 && a.lse) a.lse[orow] = (m_new + log2f(l_new)) * LN2;
    if (row_valid && r >= (un.nrows & ~7)) {
      // the last nrows % 8 rows of a clipped tile go out one by one (the rest by bulk stores)
      store_tail_row(a, sbox, sw, orow, half);
    }
    fence_async_smem();  // the producer thread's bulk store reads this tile
    mbar_arrive(c.bar(b ? BAR_OUT_RDY1 : BAR_OUT_RDY));
  }
}

template <bool PACKED, int KIND, bool DEEP, bool SPLIT>
__global__ void __launch_bounds__(THREADS, 1)
tc_attn_kernel(const __grid_constant__ TcMaps maps, const Geometry g, const AttnArgs a) {
  constexpr bool STEP = kind_is_step(KIND);
  // (PACKED: the steps of a GQA model whose block queries share tiles across heads, see decode_stream;
  // KIND: see StreamKind; DEEP: which variant of the merge role a step runs)
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const int tid = threadIdx.x;
  const int warp = tid >> 5;
  // A step reads only state that stays fixed until the next build plus what the RoPE kernel before it
  // wrote, and every global store below comes after a wait on that kernel: the next step's kernels may
  // therefore be scheduled as SMs free up (they, too, wait before their first store).  A build or a
  // full recompute writes what a following step would read early, so they do not trigger.
  if (STEP && a.step_overlap) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (a.span != nullptr && tid == 0) atomicMin(a.span, global_timer_ns());   // first CTA entry of this launch
  Cta c;
  c.base = smem_u32(smem_raw);
  c.gen = smem_raw;
  uint32_t* words = reinterpret_cast<uint32_t*>(smem_raw + SM_BAR + 8 * N_BARS);  // [0] tmem, [1] abort, [2] flag
  c.abort_flag = reinterpret_cast<volatile int*>(words + 1);
  c.flag = reinterpret_cast<volatile uint32_t*>(words + 2);
  c.status = a.status;
  // role and unit range of this CTA; the first work item is fetched before the
  // set-up below so its latency overlaps it
  const int n_ctas_merge = (int)gridDim.x - a.n_ctas_stream;
  // stream-role CTAs take the low block indices (they are scheduled first: the block
  // queries' chain of key tiles is the longest dependent chain of a step)
  const bool stream = !STEP || (int)blockIdx.x < a.n_ctas_stream;   // (only a step has fixed rows to merge)
  int first, stride, n_units;
  if (stream) {
    first = blockIdx.x; stride = a.n_ctas_stream; n_units = a.n_items * (PACKED ? a.stream_slots : g.Hq);
  } else {
    first = blockIdx.x - a.n_ctas_stream; stride = n_ctas_merge; n_units = a.n_items_merge * g.Hq;
  }
  const bool deep = !stream && DEEP;   // (DEEP: a.merge_deep, which variant of the merge role this launch runs)
  if (tid == 0) {  // descriptor fetches overlap the set-up below
    if (stream) {
      prefetch_map(STEP ? (PACKED ? &maps.q_pack : &maps.q64) : &maps.q);
      prefetch_map(&maps.k); prefetch_map(&maps.v);
    } else {
      prefetch_map(&maps.q); prefetch_map(&maps.st_o); prefetch_map(&maps.out);
      prefetch_map(deep ? &maps.k32 : &maps.k64); prefetch_map(deep ? &maps.v32 : &maps.v64);
    }
  }
  const int n_my = first < n_units ? (n_units - first + stride - 1) / stride : 0;
  WorkItem it0{};
  if (!deep && first < n_units) it0 = stream ? load_item(a.items + unit_item<PACKED, KIND>(g, a, first))
                                             : load_item(a.items_merge + first / g.Hq);
  if ((c.base & 1023u) != 0) {  // swizzled tiles need a 1024-byte aligned base
    if (tid == 0 && atomicCAS(a.status, 0, (int)LACACHE_ERR_CUDA) == 0) a.status[1] = LOC_SMEM_ALIGN;
    return;
  }
  if (deep && n_my > TC_DEEP_MAX_UNITS) {  // the host sizes launches so that the unit table never overflows
    if (tid == 0 && atomicCAS(a.status, 0, (int)LACACHE_ERR_CUDA) == 0) { a.status[1] = LOC_UNIT_TABLE; a.status[2] = n_my; }
    return;
  }
  if (tid == 0) {
    for (int i = 0; i < N_BARS; ++i) {
      uint32_t count = 1;
      if (i == BAR_P_FULL || i == BAR_P_FULL1 || i == BAR_O_FREE || i == BAR_O_FREE1 || i == BAR_EPI ||
          i == BAR_OUT_RDY || i == BAR_OUT_RDY1 || i == BAR_QC)
        count = ROW_THREADS;
      if (i == BAR_DONE) count = THREADS;
      if (i == BAR_Q_FREE && stream) count = 2;  // score MMAs done + epilogue staging read
      if (KIND == KIND_STEP2 && i == BAR_RX && stream) count = ROW_THREADS;  // the partner's row threads
      if (i >= BAR_PAIR) count = 64;
      mbar_init(c.bar(i), count);
    }
    words[1] = 0;
    words[2] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_async_smem();
  }
  if (deep) {
    // this CTA's units, read by every role from shared memory
    for (int i = tid; i < n_my; i += THREADS) {
      const int u = first + i * stride;
      // units are head-minor (unit u = row tile u / Hq of head u % Hq): a CTA's units, a
      // fixed stride apart, then cycle through the row tiles, clipped ones included
      const WorkItem w = load_item(a.items_merge + u / g.Hq);
      *reinterpret_cast<int4*>(smem_raw + DM_TAB + 16 * i) = make_int4(w.row0, w.nrows, w.blk_start, (u % g.Hq) | (w.seq << 16));
    }
  }
  __syncwarp();
  if (warp == 1) {  // (warp 1 allocates while thread 0 is still initialising the barriers)
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(words)),
                 "r"(TM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  c.tmem = words[0];
  // (paired step: nobody writes into the partner's shared memory or arrives on its barrier before the
  // partner has initialised them)
  if (KIND == KIND_STEP2) cluster_sync_all();

  if (warp == 0) {
    if (stream) {
      if (tid == 0) stream_producer<PACKED, KIND, SPLIT>(c, maps, g, a, first, stride, n_units, it0);
    } else if (deep) {
      if (tid == 0) deep_producer<SPLIT>(c, maps, g, n_my, a.k_raw != nullptr, a.out_bf16 != 0);
    } else {
      if (tid == 0) merge_producer<SPLIT>(c, maps, g, a, first, stride, n_units, it0);
    }
  } else if (warp == 1) {
    if (tid == 32) {
      if (stream) stream_mma_scores<PACKED, KIND, SPLIT>(c, g, a, first, stride, n_units, it0);
      else if (deep) deep_mma<SPLIT>(c, g, n_my, a.k_raw != nullptr);
      else merge_mma<SPLIT>(c, g, a, first, stride, n_units);
    }
  } else if (warp == 10) {
    if (tid == 320 && stream) stream_mma_pv<PACKED, KIND, SPLIT>(c, g, a, first, stride, n_units, it0);
  } else {
    if (stream) stream_rows<PACKED, KIND, SPLIT>(c, g, a, first, stride, n_units, it0);
    else if (deep) deep_rows<SPLIT>(c, g, a, n_my);
    else merge_rows(c, maps, g, a, first, stride, n_units, it0);
    bulk_wait_read();
  }
  __syncwarp();

  // teardown: free TMEM once every thread is past its last TMEM access
  if (*c.abort_flag) {
    // A bounded wait ran out and the roles have returned where they stood.  Bulk copies and tensor-core
    // products that were issued before that may still be in flight towards this CTA's shared memory and
    // TMEM: give them time to land (they take microseconds; the limit is a fixed 50 us) before both are
    // given up.
    const long long t0 = clock64();
    while (clock64() - t0 < 100000ll) {
    }
  }
  tc_fence_before();
  mbar_arrive(c.bar(BAR_DONE));
  if (warp == 1) {  // the warp that allocated
    wait_bar(c, BAR_DONE, 0, LOC_WAIT_O);
    __syncwarp();
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(c.tmem), "r"(TM_COLS) : "memory");
    // (every thread of the CTA is past its work here: BAR_DONE counts them all)
    if (a.span != nullptr && tid == 32) atomicMax(a.span + 1, global_timer_ns());   // last CTA exit
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

// rows of D features, fp32 (boxes of 32 features) or bf16 (boxes of 64): either way a box row is 128 bytes
bool make_f32_map(CUtensorMap* m, void* base, cuuint64_t d1, cuuint64_t d2, cuuint32_t b1, cuuint32_t b2, char* err,
                  int errlen, bool bf16 = false) {
  EncodeTiledFn enc = get_encode();
  if (!enc) { snprintf(err, errlen, "cuTensorMapEncodeTiled entry point not found"); return false; }
  const cuuint64_t es = bf16 ? 2 : 4;
  cuuint64_t dims[3] = {(cuuint64_t)D, d1, d2};
  cuuint64_t strides[2] = {(cuuint64_t)D * es, d1 * D * es};
  cuuint32_t box[3] = {bf16 ? 64u : 32u, b1, b2};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = enc(m, bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, base, dims, strides,
                   box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                   CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) { snprintf(err, errlen, "cuTensorMapEncodeTiled (fp32) failed with CUresult %d", (int)r); return false; }
  return true;
}

// Split-bf16 planes [plane][H][2][Tp][64] (hi plane at `base`, lo plane `plane_elems` further) as a 5-D
// tensor; fp16 values [H][2][Tp][64] as a 4-D tensor.  Box: `box_rows` rows of one head, both feature
// halves (and both planes).
bool make_qk_map(CUtensorMap* m, void* base, int H, int Tp, int box_rows, int planes, char* err, int errlen) {
  EncodeTiledFn enc = get_encode();
  if (!enc) { snprintf(err, errlen, "cuTensorMapEncodeTiled entry point not found"); return false; }
  // (with one plane the last dimension has extent 1: the same instruction loads half as much)
  cuuint64_t dims[5] = {64, (cuuint64_t)Tp, 2, (cuuint64_t)H, (cuuint64_t)planes};
  cuuint64_t strides[4] = {128, (cuuint64_t)Tp * 128, (cuuint64_t)Tp * 256, (cuuint64_t)H * Tp * 256};
  cuuint32_t box[5] = {64, (cuuint32_t)box_rows, 2, 1, (cuuint32_t)planes};
  cuuint32_t estr[5] = {1, 1, 1, 1, 1};
  CUresult r = enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, base, dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) { snprintf(err, errlen, "cuTensorMapEncodeTiled (5-D) failed with CUresult %d", (int)r); return false; }
  return true;
}
// The same planes with the head dimension inside the half dimension, so that a box of `pack` heads x
// `rows` rows lands as one [plane][half][pack * rows][64] tile.
bool make_qpack_map(CUtensorMap* m, void* base, int H, int Tp, int rows, int pack, int planes, char* err, int errlen) {
  EncodeTiledFn enc = get_encode();
  if (!enc) { snprintf(err, errlen, "cuTensorMapEncodeTiled entry point not found"); return false; }
  cuuint64_t dims[5] = {64, (cuuint64_t)Tp, (cuuint64_t)H, 2, (cuuint64_t)planes};
  cuuint64_t strides[4] = {128, (cuuint64_t)Tp * 256, (cuuint64_t)Tp * 128, (cuuint64_t)H * Tp * 256};
  cuuint32_t box[5] = {64, (cuuint32_t)rows, (cuuint32_t)pack, 2, (cuuint32_t)planes};
  cuuint32_t estr[5] = {1, 1, 1, 1, 1};
  CUresult r = enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, base, dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) { snprintf(err, errlen, "cuTensorMapEncodeTiled (packed heads) failed with CUresult %d", (int)r); return false; }
  return true;
}
bool make_v_map(CUtensorMap* m, void* base, int H, int Tp, int box_rows, char* err, int errlen) {
  EncodeTiledFn enc = get_encode();
  if (!enc) { snprintf(err, errlen, "cuTensorMapEncodeTiled entry point not found"); return false; }
  cuuint64_t dims[4] = {64, (cuuint64_t)Tp, 2, (cuuint64_t)H};
  cuuint64_t strides[3] = {128, (cuuint64_t)Tp * 128, (cuuint64_t)Tp * 256};
  cuuint32_t box[4] = {64, (cuuint32_t)box_rows, 2, 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  CUresult r = enc(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 4, base, dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) { snprintf(err, errlen, "cuTensorMapEncodeTiled (4-D) failed with CUresult %d", (int)r); return false; }
  return true;
}

}  // namespace

namespace {
// thirteen instantiations: {split planes, one plane per operand} x {build / full recompute; build over key windows; the
// step of an MHA and of a GQA model, each with either variant of the merge role}
template <bool SPLIT>
const void* const* kernel_table() {
  // (the paired step exists for one-plane operands only: with split planes the entry repeats the ordinary step)
  static const void* const t[7] = {
      (const void*)tc_attn_kernel<false, KIND_BUILD, false, SPLIT>, (const void*)tc_attn_kernel<false, KIND_WINDOW, false, SPLIT>,
      (const void*)tc_attn_kernel<false, KIND_STEP, false, SPLIT>,  (const void*)tc_attn_kernel<false, KIND_STEP, true, SPLIT>,
      (const void*)tc_attn_kernel<true, KIND_STEP, false, SPLIT>,   (const void*)tc_attn_kernel<true, KIND_STEP, true, SPLIT>,
      (const void*)tc_attn_kernel<false, SPLIT ? KIND_STEP : KIND_STEP2, true, SPLIT>};
  return t;
}
}  // namespace

cudaError_t tc_prepare() {
  for (int split = 0; split < 2; ++split) {
    const void* const* t = split ? kernel_table<true>() : kernel_table<false>();
    for (int i = 0; i < 7; ++i) {
      cudaError_t e = cudaFuncSetAttribute(t[i], cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SM_TOTAL);
      if (e != cudaSuccess) return e;
    }
  }
  return cudaSuccess;
}

bool tc_set_out(TcMaps* m, const Geometry& g, float* out, bool out_bf16, char* err, int errlen) {
  if (m->out_ptr == out) return true;
  if (!make_f32_map(&m->out, out, (cuuint64_t)g.Hq, (cuuint64_t)g.T, 1, BM, err, errlen, out_bf16)) return false;
  for (int i = 0; i < 4; ++i)
    if (!make_f32_map(&m->out_sub[i], out, (cuuint64_t)g.Hq, (cuuint64_t)g.T, 1, 64u >> i, err, errlen, out_bf16)) return false;
  m->out_ptr = out;
  return true;
}

TcMaps* tc_make_maps(const Geometry& g, const RotBuffers& rot, float* state_o, bool split, char* err, int errlen) {
  TcMaps* m = new TcMaps();
  m->out_ptr = nullptr;
  m->out = CUtensorMap{};
  // (split: the lo planes follow the hi planes at a fixed distance, see alloc_rot)
  const int planes = split ? 2 : 1;
  const int bn = tc_keys(split);
  bool ok = make_qk_map(&m->q, rot.q_hi, g.Hq, g.Tp, BM, planes, err, errlen) &&
            make_qk_map(&m->q64, rot.q_hi, g.Hq, g.Tp, 64, planes, err, errlen) &&
            // (the box always fills the 128 lanes of the tile, whose layout the MMA descriptors assume: with
            // fewer heads in a KV group than fit, the lanes past them hold other heads' rows and are ignored;
            // a model with fewer query heads than that does not pack)
            make_qpack_map(&m->q_pack, rot.q_hi, g.Hq, g.Tp, g.block_len <= 32 ? 32 : 64,
                           std::max(1, std::min(g.block_len <= 32 ? 4 : 2, g.Hq)), planes, err, errlen) &&
            make_qk_map(&m->k, rot.k_hi, g.Hkv, g.Tp, bn, planes, err, errlen) &&
            make_qk_map(&m->k64, rot.k_hi, g.Hkv, g.Tp, 64, planes, err, errlen) &&
            make_qk_map(&m->k32, rot.k_hi, g.Hkv, g.Tp, 32, planes, err, errlen) &&
            make_v_map(&m->v, rot.v, g.Hkv, g.Tp, bn, err, errlen) &&
            make_v_map(&m->v64, rot.v, g.Hkv, g.Tp, 64, err, errlen) &&
            make_v_map(&m->v32, rot.v, g.Hkv, g.Tp, 32, err, errlen) &&
            make_f32_map(&m->st_o, state_o, (cuuint64_t)g.Tp, (cuuint64_t)g.Hq, BM, 1, err, errlen);
  if (!ok) { delete m; return nullptr; }
  return m;
}

void tc_free_maps(TcMaps* m) { delete m; }

cudaError_t tc_attention(const Geometry& g, const AttnArgs& a, const TcMaps* maps, cudaStream_t s) {
  if (a.n_ctas <= 0) return cudaSuccess;
  // launched programmatically dependent on the RoPE kernel enqueued just before:
  // set-up and every load that does not depend on it overlap that kernel
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(a.n_ctas);
  cfg.blockDim = dim3(THREADS);
  cfg.dynamicSmemBytes = SM_TOTAL;
  cfg.stream = s;
  cudaLaunchAttribute attr[2];
  int n_attr = 0;
  if (!a.no_pdl) {
    attr[n_attr].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[n_attr].val.programmaticStreamSerializationAllowed = 1;
    ++n_attr;
  }
  const bool paired = a.mode == MODE_STEP && a.pair_chunks && !a.split;
  if (paired) {   // CTAs 2k and 2k + 1 form a cluster: the two key chunks of one (sequence, head)
    attr[n_attr].id = cudaLaunchAttributeClusterDimension;
    attr[n_attr].val.clusterDim.x = 2;
    attr[n_attr].val.clusterDim.y = 1;
    attr[n_attr].val.clusterDim.z = 1;
    ++n_attr;
  }
  cfg.attrs = attr;
  cfg.numAttrs = n_attr;
  const void* const* t = a.split ? kernel_table<true>() : kernel_table<false>();
  int which;
  if (a.mode != MODE_STEP) which = a.window ? 1 : 0;
  else if (paired) which = 6;
  else which = (a.pack > 1 ? 4 : 2) + (a.merge_deep ? 1 : 0);
  void* params[3] = {const_cast<TcMaps*>(maps), const_cast<Geometry*>(&g), const_cast<AttnArgs*>(&a)};
  return cudaLaunchKernelExC(&cfg, t[which], params);
}

}  // namespace lacache
