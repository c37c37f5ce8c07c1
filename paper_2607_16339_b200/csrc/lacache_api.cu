// Host side of the C ABI: context, validation, the planner that derives the
// integer metadata and the work lists, and the launch sequences.
#include <math.h>
#include <stdarg.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <algorithm>
#include <new>
#include <string>
#include <vector>

#include "lacache_internal.h"

using namespace lacache;

struct lacache_ctx {
  lacache_config cfg;
  Geometry g;
  int engine;
  std::vector<int32_t> prompt_lens, cu, seq_of_tok, pos_of_tok;
  std::vector<int32_t> blk_start_all;  // [n_blk][B]
  // work lists (offsets into d_items)
  struct ListRef { int off, n; };
  std::vector<ListRef> build_list, step_list;  // per block (step_list: SIMT all items; tcgen05 block-chunk items)
  std::vector<ListRef> merge_list;             // per block: fixed-row items of a step (tcgen05)
  // per block, tcgen05: row tiles x key windows of the incremental build (prefix state from scratch;
  // cached state = prefix state + the keys after the block; the finished block's rows from scratch;
  // every other row advanced by the finished block's keys and completed by the keys after the block)
  std::vector<ListRef> inc_prefix, inc_comb, inc_fresh, inc_fresh_chunks, inc_fused;
  // per block, tile-granular caching (Algorithm 1's overlap predicates): the build in two launches over
  // the key tiles before / after the tiles that overlap the block, the step in one
  std::vector<ListRef> tile_prefix, tile_suffix, tile_step;
  std::vector<int32_t> tile_lo_all, tile_hi_all;   // [n_blk][B]: tokens [lo, hi) of the tiles that overlap the block
  float* sample_part = nullptr;   // scratch of lacache_sample_block (allocated on first use)
  int* sample_counters = nullptr;
  StateBuffers pst{};      // prefix state of every token: its keys before the current block (allocated on first use)
  int prefix_block = -1;   // block pst is valid for
  int num_sms = 148;
  // experiment knobs, read from the environment once at create (none is needed in normal use)
  struct Knobs {
    int sc_tiles = 0;        // LACACHE_SC_TILES: key tiles per block-query chunk
    int max_ctas = 0;        // LACACHE_MAX_CTAS: cap on the persistent grid
    int stream_ctas = 0;     // LACACHE_STREAM_CTAS: role split of a step
    int deep_units = TC_DEEP_MAX_UNITS;  // LACACHE_DEEP_UNITS: units per CTA one launch of the pipelined merge variant takes
    bool no_pdl = false;     // LACACHE_NO_PDL: plain stream-ordered launches
    bool no_step_overlap = false;  // LACACHE_NO_STEP_OVERLAP
    bool no_deep = false;    // LACACHE_NO_DEEP: earlier merge variant
    bool no_qcomp = false;   // LACACHE_NO_QCOMP: no in-kernel rotation of first units
    bool no_pack = false;    // LACACHE_NO_PACK: no head packing of GQA block queries
    bool no_staged_state = false;   // LACACHE_NO_STAGED_STATE: builds store the cached state from the row threads
    bool no_pair = false;    // LACACHE_NO_PAIR: no paired CTAs (thread-block clusters) for two-chunk block rows
    bool no_chunked_advance = false;  // LACACHE_NO_CHUNKED_ADVANCE: an advance computes the finished block's rows as key-window units
    bool verbose = false;    // LACACHE_VERBOSE: prints the step plan
  } knobs;
  ListRef full_list;
  int max_chunks = 1;      // most key chunks of a step's block-row units
  std::vector<int32_t> adv_tab;   // per (block, sequence): first row and key chunks of an advance's block-row units
  int32_t* d_adv_tab = nullptr;
  int part_chunks = 1;     // chunk slots per (sequence, head) of the partial-state buffers (the advance may use more)
  std::vector<WorkItem> items_host;
  bool split = true;       // tcgen05 engine: rotated Q', K' kept as two bf16 planes (precision_mode SPLIT)

  // device memory
  std::vector<void*> allocs;
  int32_t* d_cu = nullptr;
  int32_t* d_blk_start_all = nullptr;
  int32_t* d_pos = nullptr;
  float* d_cos = nullptr;
  float* d_sin = nullptr;
  // per block: destination token and cos/sin rows of the block's B * block_len rows
  int32_t* d_blk_tok = nullptr;
  float* d_blk_cos = nullptr;
  float* d_blk_sin = nullptr;
  WorkItem* d_items = nullptr;
  RotBuffers rot{}, rot_scratch{};
  StateBuffers st{};
  float *part_m = nullptr, *part_l = nullptr, *part_o = nullptr;
  int* counters = nullptr;
  int32_t* d_status = nullptr;
  TcMaps* maps = nullptr;
  TcMaps* maps_scratch = nullptr;
  // staging for the *_host entry points
  void *hs_q = nullptr, *hs_k = nullptr, *hs_v = nullptr;       // full arrays
  void *hs_qb = nullptr, *hs_kb = nullptr, *hs_vb = nullptr;    // block arrays
  float *hs_out[2] = {nullptr, nullptr}, *hs_lse[2] = {nullptr, nullptr};   // results of alternate lacache_step_host calls
  cudaStream_t copy_stream = nullptr;     // device -> host copies of a step's result run here, beside the next step
  cudaEvent_t ev_ready[2] = {nullptr, nullptr}, ev_copied[2] = {nullptr, nullptr};
  unsigned host_steps = 0;                // lacache_step_host calls so far

  cudaEvent_t ev_start = nullptr, ev_stop = nullptr;
  unsigned long long* span_ring = nullptr;   // lacache_set_span_ring: [n_slots][2] device words
  int span_slots = 0;
  unsigned span_next = 0;
  // the role split of a step is planned once per (block, table size) and reused: a step is called
  // thousands of times per second and the host must stay ahead of the device
  struct StepPlan { int deep_cap = -1, ns = 0, pair = -1; };   // pair: every block-row item of the step has two key chunks (-1: not looked at yet)
  std::vector<StepPlan> step_plan;
  int step_overlap = 0;   // consecutive steps may overlap on the device (the caller opts in: a step then reads its inputs early)
  int steps_since_build = 0;
  int built_block = -1;
  int last_launches = 0;
  int device = 0;
  char err[512];
};

namespace {

thread_local char g_create_err[512] = "";

lacache_status fail(lacache_ctx* c, lacache_status st, const char* fmt, ...) {
  char* dst = c ? c->err : g_create_err;
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(dst, 512, fmt, ap);
  va_end(ap);
  return st;
}

#define CU_TRY(c, expr)                                                              \
  do {                                                                               \
    cudaError_t e_ = (expr);                                                         \
    if (e_ != cudaSuccess)                                                           \
      return fail(c, e_ == cudaErrorMemoryAllocation ? LACACHE_ERR_OOM : LACACHE_ERR_CUDA, \
                  "%s: %s", #expr, cudaGetErrorString(e_));                          \
  } while (0)

size_t elem_size(int dtype) { return dtype == LACACHE_DTYPE_BF16 ? 2 : 4; }

bool misaligned(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; }

template <class T>
cudaError_t dev_alloc(lacache_ctx* c, T** p, size_t n_elems, bool zero = false) {
  void* q = nullptr;
  size_t bytes = std::max<size_t>(n_elems * sizeof(T), 256);
  cudaError_t e = cudaMalloc(&q, bytes);
  if (e != cudaSuccess) return e;
  c->allocs.push_back(q);
  if (zero) {
    e = cudaMemset(q, 0, bytes);
    if (e != cudaSuccess) return e;
  }
  *p = reinterpret_cast<T*>(q);
  return cudaSuccess;
}

// Tiles of `rows_per_item` query rows over [lo, hi) of one sequence.
void add_row_tiles(std::vector<WorkItem>& v, int seq, int lo, int hi, int rows_per_item, int seq_start,
                   int seq_end, int blk_start, int kind = ITEM_ROWS) {
  for (int r = lo; r < hi; r += rows_per_item) {
    WorkItem w{};
    w.kind = kind;
    w.seq = seq;
    w.row0 = r;
    w.nrows = std::min(rows_per_item, hi - r);
    w.pad = 1;
    w.seq_start = seq_start;
    w.seq_end = seq_end;
    w.blk_start = blk_start;
    v.push_back(w);
  }
}

lacache_status alloc_rot(lacache_ctx* c, RotBuffers* r) {
  const Geometry& g = c->g;
  size_t nq = (size_t)g.Hq * g.Tp * g.d, nk = (size_t)g.Hkv * g.Tp * g.d;
  if (c->engine == LACACHE_ENGINE_TCGEN05) {
    // hi and lo planes of a tensor share one allocation (the lo plane starts
    // right after the hi plane): the tensor maps address them as one 5-D tensor
    // (plain operands: no lo plane at all)
    uint16_t *a, *cc, *e;
    const size_t planes = c->split ? 2 : 1;
    CU_TRY(c, dev_alloc(c, &a, planes * nq, true));
    CU_TRY(c, dev_alloc(c, &cc, planes * nk, true));
    CU_TRY(c, dev_alloc(c, &e, nk, true));
    *r = RotBuffers{a, c->split ? a + nq : nullptr, cc, c->split ? cc + nk : nullptr, e};
  } else {
    float *a, *b, *cc;
    CU_TRY(c, dev_alloc(c, &a, nq, true));
    CU_TRY(c, dev_alloc(c, &b, nk, true));
    CU_TRY(c, dev_alloc(c, &cc, nk, true));
    *r = RotBuffers{a, nullptr, b, nullptr, cc};
  }
  return LACACHE_OK;
}

lacache_status create_impl(const lacache_config* cfg, lacache_ctx* c) {
  c->cfg = *cfg;
  c->cfg.prompt_lens = nullptr;
  c->err[0] = 0;
  {
    lacache_ctx::Knobs& k = c->knobs;
    auto geti = [](const char* name, int dflt) { const char* e = getenv(name); return e ? atoi(e) : dflt; };
    k.sc_tiles = geti("LACACHE_SC_TILES", 0);
    k.max_ctas = geti("LACACHE_MAX_CTAS", 0);
    k.stream_ctas = geti("LACACHE_STREAM_CTAS", 0);
    k.deep_units = std::max(1, std::min(geti("LACACHE_DEEP_UNITS", TC_DEEP_MAX_UNITS), (int)TC_DEEP_MAX_UNITS));
    k.no_pdl = getenv("LACACHE_NO_PDL") != nullptr;
    k.no_step_overlap = getenv("LACACHE_NO_STEP_OVERLAP") != nullptr;
    k.no_deep = getenv("LACACHE_NO_DEEP") != nullptr;
    k.no_qcomp = getenv("LACACHE_NO_QCOMP") != nullptr;
    k.no_pack = getenv("LACACHE_NO_PACK") != nullptr;
    k.no_pair = getenv("LACACHE_NO_PAIR") != nullptr;
    k.no_staged_state = getenv("LACACHE_NO_STAGED_STATE") != nullptr;
    k.no_chunked_advance = getenv("LACACHE_NO_CHUNKED_ADVANCE") != nullptr;
    k.verbose = getenv("LACACHE_VERBOSE") != nullptr;
  }
  if (cfg->batch < 1 || !cfg->prompt_lens) return fail(c, LACACHE_ERR_INVALID_ARG, "batch < 1 or prompt_lens NULL");
  if (cfg->dtype != LACACHE_DTYPE_BF16 && cfg->dtype != LACACHE_DTYPE_FP32)
    return fail(c, LACACHE_ERR_UNSUPPORTED, "dtype %d", cfg->dtype);
  if (cfg->head_dim != 64 && cfg->head_dim != 128)
    return fail(c, LACACHE_ERR_UNSUPPORTED, "head_dim %d (64 or 128)", cfg->head_dim);
  if (cfg->n_q_heads < 1 || cfg->n_kv_heads < 1 || cfg->n_q_heads % cfg->n_kv_heads)
    return fail(c, LACACHE_ERR_SHAPE, "n_q_heads %d not a multiple of n_kv_heads %d", cfg->n_q_heads,
                cfg->n_kv_heads);
  if (cfg->gen_len < 1 || cfg->block_len < 1 || cfg->gen_len % cfg->block_len)
    return fail(c, LACACHE_ERR_SHAPE, "gen_len %d not a positive multiple of block_len %d", cfg->gen_len,
                cfg->block_len);
  if (!(cfg->rope_theta > 0.f)) return fail(c, LACACHE_ERR_INVALID_ARG, "rope_theta must be > 0");
  for (int b = 0; b < cfg->batch; ++b)
    if (cfg->prompt_lens[b] < 0) return fail(c, LACACHE_ERR_SHAPE, "prompt_lens[%d] < 0", b);

  if (cfg->out_dtype != LACACHE_OUT_BF16 && cfg->out_dtype != LACACHE_OUT_FP32)
    return fail(c, LACACHE_ERR_INVALID_ARG, "out_dtype %d", cfg->out_dtype);
  if (cfg->precision_mode != LACACHE_PRECISION_PLAIN && cfg->precision_mode != LACACHE_PRECISION_SPLIT &&
      cfg->precision_mode != LACACHE_PRECISION_FP16)
    return fail(c, LACACHE_ERR_UNSUPPORTED, "precision_mode %d (0 = one bf16 plane per operand, 1 = split bf16 planes, 3 = one fp16 plane)", cfg->precision_mode);
  if (cfg->cache_granularity != LACACHE_GRANULARITY_TOKEN && cfg->cache_granularity != LACACHE_GRANULARITY_TILE)
    return fail(c, LACACHE_ERR_INVALID_ARG, "cache_granularity %d", cfg->cache_granularity);
  bool tc_ok = cfg->dtype == LACACHE_DTYPE_BF16 && cfg->head_dim == 128 && cfg->block_len <= TC_MAX_BLOCK;
  if (cfg->engine == LACACHE_ENGINE_AUTO) c->engine = tc_ok ? LACACHE_ENGINE_TCGEN05 : LACACHE_ENGINE_SIMT;
  else if (cfg->engine == LACACHE_ENGINE_SIMT) c->engine = LACACHE_ENGINE_SIMT;
  else if (cfg->engine == LACACHE_ENGINE_TCGEN05) {
    if (!tc_ok) return fail(c, LACACHE_ERR_UNSUPPORTED, "tcgen05 engine needs bf16, head_dim 128, block_len <= 64");
    c->engine = LACACHE_ENGINE_TCGEN05;
  } else return fail(c, LACACHE_ERR_INVALID_ARG, "engine %d", cfg->engine);
  if (cfg->cache_granularity == LACACHE_GRANULARITY_TILE && c->engine != LACACHE_ENGINE_TCGEN05)
    return fail(c, LACACHE_ERR_UNSUPPORTED, "tile-granular caching needs the tcgen05 engine (bf16, head_dim 128, block_len <= 64)");

  // ---- integer metadata (index sets of Sec. 3.3.1) ----
  Geometry& g = c->g;
  g.B = cfg->batch;
  c->prompt_lens.assign(cfg->prompt_lens, cfg->prompt_lens + g.B);
  c->cu.assign(g.B + 1, 0);
  g.maxN = 0;
  long long tot = 0;
  for (int b = 0; b < g.B; ++b) {
    int n = c->prompt_lens[b] + cfg->gen_len;
    tot += n;
    if (tot > (1ll << 30)) return fail(c, LACACHE_ERR_SHAPE, "too many tokens");
    c->cu[b + 1] = (int32_t)tot;
    g.maxN = std::max(g.maxN, n);
  }
  g.T = (int)tot;
  g.Tp = (g.T + 127) / 128 * 128 + 128;
  g.Hq = cfg->n_q_heads; g.Hkv = cfg->n_kv_heads; g.d = cfg->head_dim; g.group = g.Hq / g.Hkv;
  g.gen_len = cfg->gen_len; g.block_len = cfg->block_len; g.n_blk = cfg->gen_len / cfg->block_len;
  double scale = cfg->softmax_scale > 0.f ? (double)cfg->softmax_scale : 1.0 / sqrt((double)g.d);
  g.scale_log2 = (float)(scale * 1.4426950408889634074);
  c->seq_of_tok.resize(g.T);
  c->pos_of_tok.resize(g.T);
  for (int b = 0; b < g.B; ++b)
    for (int t = c->cu[b]; t < c->cu[b + 1]; ++t) { c->seq_of_tok[t] = b; c->pos_of_tok[t] = t - c->cu[b]; }
  c->blk_start_all.resize((size_t)g.n_blk * g.B);
  for (int k = 0; k < g.n_blk; ++k)
    for (int b = 0; b < g.B; ++b) c->blk_start_all[(size_t)k * g.B + b] = c->cu[b] + c->prompt_lens[b] + k * g.block_len;

  // ---- device (queried before planning: the cost models below size work for its SM count) ----
  CU_TRY(c, cudaGetDevice(&c->device));
  cudaDeviceProp prop;
  CU_TRY(c, cudaGetDeviceProperties(&prop, c->device));
  c->num_sms = prop.multiProcessorCount;
  if (c->knobs.max_ctas > 0) c->num_sms = std::max(1, std::min(c->num_sms, c->knobs.max_ctas));
  if (c->engine == LACACHE_ENGINE_TCGEN05 && prop.major != 10)
    return fail(c, LACACHE_ERR_UNSUPPORTED, "tcgen05 engine needs an sm_100 device, found sm_%d%d", prop.major, prop.minor);

  // ---- work lists ----
  const bool tc = c->engine == LACACHE_ENGINE_TCGEN05;
  c->split = cfg->precision_mode == LACACHE_PRECISION_SPLIT;
  c->g.op_f16 = (c->engine == LACACHE_ENGINE_TCGEN05 && cfg->precision_mode == LACACHE_PRECISION_FP16) ? 1 : 0;
  const int TC_KEYS = tc_keys(c->split);
  const int R = tc ? TC_ROWS : SIMT_ROWS;
  std::vector<WorkItem> items;
  // Block-query units: the keys of each (sequence, head) are cut into balanced
  // chunks of `tpc` tiles.  Unless the caller fixes it, pick the chunk size and
  // the role split together from a small cost model (times in microseconds,
  // measured on B200: a stream unit costs ~3 + 1.6 per key tile, plus ~2 + 0.8
  // per chunk when partial states have to be merged; a merge unit ~2.6
  // (pipelined variant, block_len <= 32, few units per CTA) or ~3.4 after a ~4 us cold start),
  // at most 16 chunks per sequence.
  int tpc = cfg->sc_tiles_per_chunk;
  if (c->knobs.sc_tiles > 0) tpc = c->knobs.sc_tiles;
  if (tc && tpc <= 0) {
    int max_nkt = 1;
    long long rows_u = 0;
    for (int b = 0; b < g.B; ++b) {
      max_nkt = std::max(max_nkt, (c->cu[b + 1] - c->cu[b] + TC_KEYS - 1) / TC_KEYS);
      int n_u = c->cu[b + 1] - c->cu[b] - g.block_len;
      rows_u += (n_u + TC_ROWS - 1) / TC_ROWS + 1;
    }
    const int sms = c->num_sms;
    const double units_m = (double)rows_u * g.Hq;
    double best = 1e30;
    for (int cand = 1; cand <= max_nkt; ++cand) {
      // the chunks this candidate would produce (balanced within a sequence, as below); a CTA
      // draws short and long units alike, so a unit is costed between the mean and the longest
      double units_s = 0, sum_t = 0;
      int max_ch = 1, max_t = 1;
      for (int b = 0; b < g.B; ++b) {
        int nkt = (c->cu[b + 1] - c->cu[b] + TC_KEYS - 1) / TC_KEYS;
        int ch = std::min(16, (nkt + cand - 1) / cand);
        int per = (nkt + ch - 1) / ch;
        ch = (nkt + per - 1) / per;
        max_ch = std::max(max_ch, ch);
        max_t = std::max(max_t, per);
        units_s += ch * (double)g.Hq;
        sum_t += nkt;
      }
      const double eff_tiles = 0.5 * (sum_t * g.Hq / units_s + max_t);
      const double merge_cost = max_ch > 1 ? 2.0 + 0.8 * max_ch : 0.0;
      for (int ns = std::min(8, std::max(1, sms / 4)); ns <= std::max(1, sms - 8); ns += 4) {
        double ts = ceil(units_s / ns) * (3.0 + 1.6 * eff_tiles + merge_cost);
        // (a CTA with many merge units runs in the HBM-saturated regime, where a unit costs more)
        const double per_cta = ceil(units_m / (sms - ns));
        double tm = 4.0 + per_cta * ((g.block_len <= 32 && per_cta <= 8) ? 2.6 : 3.4);
        double t = std::max(ts, tm);
        if (t < best - 1e-9) { best = t; tpc = cand; }
      }
    }
  }
  if (tpc <= 0) tpc = 2;
  c->max_chunks = 1;
  for (int k = 0; k < g.n_blk; ++k) {
    int off = (int)items.size();
    // block-query items
    for (int b = 0; b < g.B; ++b) {
      int bs = c->blk_start_all[(size_t)k * g.B + b];
      if (tc) {
        int n = c->cu[b + 1] - c->cu[b];
        int nkt = (n + TC_KEYS - 1) / TC_KEYS;
        int chunks = std::min(16, (nkt + tpc - 1) / tpc);
        int tpc_b = (nkt + chunks - 1) / chunks;       // balanced
        chunks = (nkt + tpc_b - 1) / tpc_b;
        c->max_chunks = std::max(c->max_chunks, chunks);
        for (int ch = 0; ch < chunks; ++ch) {
          WorkItem w{};
          w.kind = ITEM_BLOCK_CHUNK; w.seq = b; w.row0 = bs; w.nrows = g.block_len;
          w.chunk = ch; w.kt0 = ch * tpc_b; w.kt1 = std::min(nkt, (ch + 1) * tpc_b);
          w.pad = chunks;
          w.seq_start = c->cu[b]; w.seq_end = c->cu[b + 1]; w.blk_start = bs;
          items.push_back(w);
        }
      } else {
        add_row_tiles(items, b, bs, bs + g.block_len, R, c->cu[b], c->cu[b + 1], bs, ITEM_BLOCK_CHUNK);
      }
    }
    int rows_off = (int)items.size();
    for (int b = 0; b < g.B; ++b) {
      int bs = c->blk_start_all[(size_t)k * g.B + b];
      add_row_tiles(items, b, c->cu[b], bs, R, c->cu[b], c->cu[b + 1], bs);
      add_row_tiles(items, b, bs + g.block_len, c->cu[b + 1], R, c->cu[b], c->cu[b + 1], bs);
    }
    if (tc) {
      c->step_list.push_back({off, rows_off - off});
      c->merge_list.push_back({rows_off, (int)items.size() - rows_off});
    } else {
      c->step_list.push_back({off, (int)items.size() - off});
      c->merge_list.push_back({0, 0});
    }
    c->build_list.push_back({rows_off, (int)items.size() - rows_off});
  }
  int inc_chunks = 1;
  c->adv_tab.assign((size_t)g.n_blk * g.B * 2, 0);
  for (int k = 0; k < g.n_blk && tc; ++k) {
    // Incremental build.  With s the block's first token and e one past its last, of a sequence
    // [cs, ce): the prefix state holds keys [cs, s); the cached state adds keys [e, ce); advancing
    // from block k - 1 adds that block's keys [s - L_b, s) to the rows outside it and computes the
    // rows inside it (whose queries changed) over [cs, s) from scratch.
    auto window = [&](int from, int base, int k0, int k1, int flags) {
      for (size_t i = from; i < items.size(); ++i) {
        items[i].kind = ITEM_ROWS_WINDOW;
        items[i].pad = base;
        items[i].kt0 = k0;
        items[i].kt1 = k1;
        items[i].chunk = flags;
      }
    };
    enum { W_INIT = 1, W_SNAP = 2, W_SKIP_BLOCK = 4, W_JUMP_BLOCK = 8 };
    int off = (int)items.size();
    for (int b = 0; b < g.B; ++b) {
      const int cs = c->cu[b], ce = c->cu[b + 1], s0 = c->blk_start_all[(size_t)k * g.B + b], e0 = s0 + g.block_len;
      const int from = (int)items.size();
      add_row_tiles(items, b, cs, s0, R, cs, ce, s0);
      add_row_tiles(items, b, e0, ce, R, cs, ce, s0);
      window(from, cs, cs, s0, 0);
    }
    c->inc_prefix.push_back({off, (int)items.size() - off});
    off = (int)items.size();
    for (int b = 0; b < g.B; ++b) {
      const int cs = c->cu[b], ce = c->cu[b + 1], s0 = c->blk_start_all[(size_t)k * g.B + b], e0 = s0 + g.block_len;
      const int from = (int)items.size();
      add_row_tiles(items, b, cs, s0, R, cs, ce, s0);
      add_row_tiles(items, b, e0, ce, R, cs, ce, s0);
      window(from, e0, e0, ce, W_INIT);
    }
    c->inc_comb.push_back({off, (int)items.size() - off});
    // advancing from block k - 1 (rows [sp, s0), blocks are consecutive), in two launches:
    off = (int)items.size();
    for (int b = 0; b < g.B && k > 0; ++b) {
      // its rows changed their queries: prefix state over every key before block k, from scratch
      const int cs = c->cu[b], ce = c->cu[b + 1], s0 = c->blk_start_all[(size_t)k * g.B + b];
      const int from = (int)items.size();
      add_row_tiles(items, b, s0 - g.block_len, s0, R, cs, ce, s0);
      window(from, cs, cs, s0, 0);
    }
    c->inc_fresh.push_back({off, (int)items.size() - off});
    // the same rows as block-row units of the step kernel, their keys [cs, s0) cut into chunks that
    // spread over the SMs (a handful of row tiles otherwise walk the whole prefix one after the other)
    off = (int)items.size();
    for (int b = 0; b < g.B && k > 0; ++b) {
      const int cs = c->cu[b], s0 = c->blk_start_all[(size_t)k * g.B + b];
      const int nkt = (s0 - cs + TC_KEYS - 1) / TC_KEYS;
      // (units of all sequences: one per sequence and head, or per packed group of heads; at most eight
      // chunks, which the last one to arrive merges with every load in flight at once)
      const int fit = 128 / (g.block_len <= 32 ? 32 : 64);
      const int pack = (g.group >= 2 && g.Hq >= fit && !c->knobs.no_pack) ? std::min(fit, g.group) : 1;
      const int slots = g.B * g.Hkv * ((g.group + pack - 1) / pack);
      int chunks = std::max(1, std::min({8, nkt, c->num_sms / slots}));
      const int per = (nkt + chunks - 1) / chunks;
      chunks = (nkt + per - 1) / per;
      inc_chunks = std::max(inc_chunks, chunks);
      c->adv_tab[((size_t)k * g.B + b) * 2] = s0 - g.block_len;
      c->adv_tab[((size_t)k * g.B + b) * 2 + 1] = chunks;
      for (int ch = 0; ch < chunks; ++ch) {
        WorkItem w{};
        w.kind = ITEM_BLOCK_CHUNK; w.seq = b; w.row0 = s0 - g.block_len; w.nrows = g.block_len;
        w.chunk = ch; w.kt0 = ch * per; w.kt1 = std::min(nkt, (ch + 1) * per);
        w.pad = chunks;
        w.seq_start = cs; w.seq_end = s0;       // (the end of the key range, not of the sequence)
        w.blk_start = s0 - g.block_len;
        items.push_back(w);
      }
    }
    c->inc_fresh_chunks.push_back({off, (int)items.size() - off});
    off = (int)items.size();
    for (int b = 0; b < g.B && k > 0; ++b) {
      const int cs = c->cu[b], ce = c->cu[b + 1], s0 = c->blk_start_all[(size_t)k * g.B + b], e0 = s0 + g.block_len;
      const int sp = s0 - g.block_len;
      // every other fixed row: old prefix state + the finished block's keys (exactly the first key
      // tile, which ends at s0) = new prefix state, stored; + the keys after block k = cached state
      int from = (int)items.size();
      add_row_tiles(items, b, cs, sp, R, cs, ce, s0);
      add_row_tiles(items, b, e0, ce, R, cs, ce, s0);
      window(from, s0 - TC_KEYS, sp, ce > e0 ? ce : s0, W_INIT | W_SNAP | W_JUMP_BLOCK);
      // the finished block's rows: their new prefix state + the keys after block k
      from = (int)items.size();
      add_row_tiles(items, b, sp, s0, R, cs, ce, s0);
      window(from, e0, e0, ce, W_INIT);
    }
    c->inc_fused.push_back({off, (int)items.size() - off});
  }
  c->part_chunks = std::max(c->max_chunks, inc_chunks);
  if (cfg->cache_granularity == LACACHE_GRANULARITY_TILE) {
    // Algorithm 1 at tile granularity, tiles of TC_ROWS tokens counted from the start of each sequence
    // (B_r = B_c).  With [lo, hi) the tokens of the tiles that overlap the block: state is cached for the
    // rows outside [lo, hi) over the keys outside [lo, hi) (first the keys before lo, then, on top, the
    // keys from hi on); a step gives those rows the keys [lo, hi) and runs the rows of [lo, hi) over all
    // keys.  The work items are key-window items of the build kernel.
    enum { W_INIT = 1, W_OUT = 16 };
    auto window = [&](size_t from, int base, int k0, int k1, int flags) {
      for (size_t i = from; i < items.size(); ++i) {
        items[i].kind = ITEM_ROWS_WINDOW;
        items[i].pad = base;
        items[i].kt0 = k0;
        items[i].kt1 = k1;
        items[i].chunk = flags;
      }
    };
    c->tile_lo_all.resize((size_t)g.n_blk * g.B);
    c->tile_hi_all.resize((size_t)g.n_blk * g.B);
    for (int k = 0; k < g.n_blk; ++k) {
      for (int pass = 0; pass < 3; ++pass) {
        const int off = (int)items.size();
        for (int b = 0; b < g.B; ++b) {
          const int cs = c->cu[b], ce = c->cu[b + 1], s0 = c->blk_start_all[(size_t)k * g.B + b], e0 = s0 + g.block_len;
          const int lo = cs + (s0 - cs) / TC_ROWS * TC_ROWS;
          const int hi = std::min(ce, cs + (e0 - cs + TC_ROWS - 1) / TC_ROWS * TC_ROWS);
          c->tile_lo_all[(size_t)k * g.B + b] = lo;
          c->tile_hi_all[(size_t)k * g.B + b] = hi;
          size_t from = items.size();
          if (pass == 2) {   // the rows of the overlapping tiles x all keys: the longest units, so they go first
            add_row_tiles(items, b, lo, hi, R, cs, ce, s0);
            window(from, cs, cs, ce, W_OUT);
            from = items.size();
          }
          // (no unit without keys: a sequence with nothing before the overlapping tiles starts its state in
          // the second launch, one with nothing after them is complete after the first)
          if (pass == 0 && lo == cs) continue;
          if (pass == 1 && hi == ce) continue;
          add_row_tiles(items, b, cs, lo, R, cs, ce, s0);
          add_row_tiles(items, b, hi, ce, R, cs, ce, s0);
          if (pass == 0) window(from, cs, cs, lo, 0);
          else if (pass == 1) window(from, hi, hi, ce, lo > cs ? W_INIT : 0);
          else window(from, lo, lo, hi, W_INIT | W_OUT);
        }
        (pass == 0 ? c->tile_prefix : pass == 1 ? c->tile_suffix : c->tile_step).push_back({off, (int)items.size() - off});
      }
    }
  }
  {
    int off = (int)items.size();
    for (int b = 0; b < g.B; ++b) add_row_tiles(items, b, c->cu[b], c->cu[b + 1], R, c->cu[b], c->cu[b + 1], 0);
    c->full_list = {off, (int)items.size() - off};
  }
  c->items_host = items;

  // ---- device memory ----
  CU_TRY(c, simt_prepare());
  if (tc) CU_TRY(c, tc_prepare());

  CU_TRY(c, dev_alloc(c, &c->d_cu, g.B + 1));
  CU_TRY(c, cudaMemcpy(c->d_cu, c->cu.data(), sizeof(int32_t) * (g.B + 1), cudaMemcpyHostToDevice));
  CU_TRY(c, dev_alloc(c, &c->d_blk_start_all, c->blk_start_all.size()));
  CU_TRY(c, cudaMemcpy(c->d_blk_start_all, c->blk_start_all.data(), sizeof(int32_t) * c->blk_start_all.size(), cudaMemcpyHostToDevice));
  CU_TRY(c, dev_alloc(c, &c->d_pos, g.T));
  CU_TRY(c, cudaMemcpy(c->d_pos, c->pos_of_tok.data(), sizeof(int32_t) * g.T, cudaMemcpyHostToDevice));
  CU_TRY(c, dev_alloc(c, &c->d_adv_tab, c->adv_tab.size()));
  CU_TRY(c, cudaMemcpy(c->d_adv_tab, c->adv_tab.data(), sizeof(int32_t) * c->adv_tab.size(), cudaMemcpyHostToDevice));
  CU_TRY(c, dev_alloc(c, &c->d_items, items.size()));
  CU_TRY(c, cudaMemcpy(c->d_items, items.data(), sizeof(WorkItem) * items.size(), cudaMemcpyHostToDevice));
  {
    // cos/sin of p * theta^(-2c/d), evaluated in double, stored as fp32 (Eq. 1)
    int half = g.d / 2;
    std::vector<float> cs((size_t)g.maxN * half), sn((size_t)g.maxN * half);
    for (int cidx = 0; cidx < half; ++cidx) {
      double f = pow((double)cfg->rope_theta, -2.0 * (double)cidx / (double)g.d);
      for (int p = 0; p < g.maxN; ++p) {
        double ang = (double)p * f;
        cs[(size_t)p * half + cidx] = (float)cos(ang);
        sn[(size_t)p * half + cidx] = (float)sin(ang);
      }
    }
    CU_TRY(c, dev_alloc(c, &c->d_cos, cs.size()));
    CU_TRY(c, dev_alloc(c, &c->d_sin, sn.size()));
    CU_TRY(c, cudaMemcpy(c->d_cos, cs.data(), sizeof(float) * cs.size(), cudaMemcpyHostToDevice));
    CU_TRY(c, cudaMemcpy(c->d_sin, sn.data(), sizeof(float) * sn.size(), cudaMemcpyHostToDevice));
    // the same rows gathered per block row (row r of block k: sequence r / block_len,
    // offset r % block_len), so the step's RoPE kernel needs no dependent look-ups
    const size_t rows = (size_t)g.n_blk * g.B * g.block_len;
    std::vector<int32_t> btok(rows);
    std::vector<float> bcs(rows * half), bsn(rows * half);
    for (int k = 0; k < g.n_blk; ++k)
      for (int r = 0; r < g.B * g.block_len; ++r) {
        const size_t row = (size_t)k * g.B * g.block_len + r;
        const int tok = c->blk_start_all[(size_t)k * g.B + r / g.block_len] + r % g.block_len;
        const int pos = c->pos_of_tok[tok];
        btok[row] = tok;
        std::copy(cs.begin() + (size_t)pos * half, cs.begin() + (size_t)(pos + 1) * half, bcs.begin() + row * half);
        std::copy(sn.begin() + (size_t)pos * half, sn.begin() + (size_t)(pos + 1) * half, bsn.begin() + row * half);
      }
    CU_TRY(c, dev_alloc(c, &c->d_blk_tok, rows));
    CU_TRY(c, dev_alloc(c, &c->d_blk_cos, rows * half));
    CU_TRY(c, dev_alloc(c, &c->d_blk_sin, rows * half));
    CU_TRY(c, cudaMemcpy(c->d_blk_tok, btok.data(), sizeof(int32_t) * rows, cudaMemcpyHostToDevice));
    CU_TRY(c, cudaMemcpy(c->d_blk_cos, bcs.data(), sizeof(float) * bcs.size(), cudaMemcpyHostToDevice));
    CU_TRY(c, cudaMemcpy(c->d_blk_sin, bsn.data(), sizeof(float) * bsn.size(), cudaMemcpyHostToDevice));
  }
  lacache_status st = alloc_rot(c, &c->rot);
  if (st != LACACHE_OK) return st;
  st = alloc_rot(c, &c->rot_scratch);
  if (st != LACACHE_OK) return st;
  CU_TRY(c, dev_alloc(c, &c->st.m, (size_t)g.Hq * g.Tp, true));
  CU_TRY(c, dev_alloc(c, &c->st.l, (size_t)g.Hq * g.Tp, true));
  CU_TRY(c, dev_alloc(c, &c->st.o, (size_t)g.Hq * g.Tp * g.d, true));
  size_t nparts = (size_t)g.B * g.Hq * c->part_chunks * g.block_len;
  CU_TRY(c, dev_alloc(c, &c->part_m, nparts));
  CU_TRY(c, dev_alloc(c, &c->part_l, nparts));
  CU_TRY(c, dev_alloc(c, &c->part_o, nparts * g.d));
  CU_TRY(c, dev_alloc(c, &c->counters, (size_t)g.B * g.Hq, true));
  CU_TRY(c, dev_alloc(c, &c->d_status, 4, true));
  if (tc) {
    c->maps = tc_make_maps(g, c->rot, c->st.o, c->split, c->err, sizeof(c->err));
    if (!c->maps) return LACACHE_ERR_CUDA;
    c->maps_scratch = tc_make_maps(g, c->rot_scratch, c->st.o, c->split, c->err, sizeof(c->err));
    if (!c->maps_scratch) return LACACHE_ERR_CUDA;
  }
  CU_TRY(c, cudaDeviceSynchronize());
  return LACACHE_OK;
}

void destroy_impl(lacache_ctx* c) {
  cudaDeviceSynchronize();
  for (void* p : c->allocs) cudaFree(p);
  for (int b = 0; b < 2; ++b) {
    if (c->ev_ready[b]) cudaEventDestroy(c->ev_ready[b]);
    if (c->ev_copied[b]) cudaEventDestroy(c->ev_copied[b]);
  }
  if (c->copy_stream) cudaStreamDestroy(c->copy_stream);
  if (c->maps) tc_free_maps(c->maps);
  if (c->maps_scratch) tc_free_maps(c->maps_scratch);
  delete c;
}

// Units per CTA the pipelined merge variant takes in one launch (its table size; the
// LACACHE_DEEP_UNITS knob lowers it so that small cases exercise the multi-launch path).
int deep_unit_cap(const lacache_ctx* c) { return c->knobs.deep_units; }

// block queries of a GQA model: heads of one KV group side by side in the 128 lanes of a tile
void set_packing(lacache_ctx* c, AttnArgs& a) {
  if (c->g.group < 2 || c->knobs.no_pack) return;
  const int rows = c->g.block_len <= 32 ? 32 : 64;
  const int pack = std::min(128 / rows, c->g.group);
  if (c->g.Hq < 128 / rows) return;   // the packed tile's load takes 128 / rows heads at a time
  if (pack >= 2) {
    a.pack = pack; a.pack_rows = rows;
    a.stream_slots = c->g.Hkv * ((c->g.group + pack - 1) / pack);
  }
}

AttnArgs attn_args(lacache_ctx* c, int mode, lacache_ctx::ListRef list, int blk, const RotBuffers& rot,
                   float* out, float* lse) {
  AttnArgs a{};
  a.mode = mode;
  a.items = c->d_items + list.off;
  a.n_items = list.n;
  a.cu = c->d_cu;
  a.blk_start = blk >= 0 ? c->d_blk_start_all + (size_t)blk * c->g.B : nullptr;
  a.rot = rot;
  a.st = c->st;
  a.out = out;
  a.lse = lse;
  a.out_bf16 = c->cfg.out_dtype == LACACHE_OUT_BF16 ? 1 : 0;
  a.part_m = c->part_m; a.part_l = c->part_l; a.part_o = c->part_o;
  a.counters = c->counters;
  a.max_chunks = c->part_chunks;
  a.status = c->d_status;
  a.no_pdl = c->knobs.no_pdl ? 1 : 0;
  a.split = c->split ? 1 : 0;
  if (c->engine == LACACHE_ENGINE_TCGEN05) {
    // persistent grid: one CTA per SM, split between the two roles by a cost
    // estimate (units x per-unit cost, in arbitrary time units)
    const int Hq = c->g.Hq;
    a.stream_slots = Hq; a.pack = 1; a.pack_rows = 0;
    if (mode == MODE_STEP) set_packing(c, a);
    long long units_stream = (long long)list.n * a.stream_slots;
    if (mode == MODE_STEP) {
      lacache_ctx::ListRef ml = c->merge_list[blk];
      a.items_merge = c->d_items + ml.off;
      a.n_items_merge = ml.n;
      long long units_merge = (long long)ml.n * Hq;
      int total = (int)std::min<long long>(c->num_sms, units_stream + units_merge);
      const bool deep_ok = c->g.block_len <= 32 && !c->knobs.no_deep;
      const int deep_cap = deep_unit_cap(c);
      if (c->step_plan.empty()) c->step_plan.resize(c->g.n_blk);
      lacache_ctx::StepPlan& plan = c->step_plan[blk];
      const bool planned = plan.deep_cap == deep_cap;
      double sum_tiles = 0;   // ragged batches mix short and long units on a CTA: cost a unit between mean and longest
      int longest = 1;
      for (int i = 0; i < list.n && !planned; ++i) {
        const WorkItem& w = c->items_host[list.off + i];
        sum_tiles += w.kt1 - w.kt0;
        longest = std::max(longest, w.kt1 - w.kt0);
      }
      const double max_tiles = list.n > 0 ? 0.5 * (sum_tiles / list.n + longest) : 1.0;
      int ns = planned ? plan.ns : 1;
      double best = 1e30;
      for (int cand = 1; cand < total && !planned; ++cand) {
        double ts = ceil((double)units_stream / cand) * (3.0 + 1.6 * max_tiles + (c->max_chunks > 1 ? 2.0 + 0.8 * c->max_chunks : 0.0));
        double per_cta = ceil((double)units_merge / (total - cand));
        double rest = 0.0;   // merge units beyond what one launch of the pipelined variant takes: further launches, all SMs
        if (deep_ok && per_cta > deep_cap) {
          rest = (double)units_merge - (double)deep_cap * (total - cand);
          per_cta = deep_cap;
        }
        double tm = 4.0 + per_cta * ((c->g.block_len <= 32 && per_cta <= 8) ? 2.6 : 3.4);
        double t = std::max(ts, tm) + (rest > 0 ? 4.0 + ceil(rest / c->num_sms) * 3.4 : 0.0);
        if (t < best - 1e-9) { best = t; ns = cand; }
      }
      if (c->knobs.stream_ctas > 0) ns = c->knobs.stream_ctas;
      if (units_merge == 0) ns = total;
      else ns = std::max(1, std::min(ns, total - 1));
      ns = (int)std::min<long long>(ns, units_stream);
      plan.deep_cap = deep_cap;
      plan.ns = ns;
      a.n_ctas_stream = ns;
      if (c->knobs.verbose) {
        static int printed = 0;
        if (printed++ < 16) fprintf(stderr, "lacache: step plan (block %d): %lld stream units (max %d chunks), %lld merge units, %d stream CTAs of %d\n", blk, units_stream, c->max_chunks, units_merge, ns, total);
      }
      a.n_ctas = ns + (int)std::min<long long>(units_merge, std::max(0, c->num_sms - ns));
      {
        const int n_merge_ctas = a.n_ctas - ns;
        const long long per_cta = n_merge_ctas > 0 ? (units_merge + n_merge_ctas - 1) / n_merge_ctas : 0;
        a.merge_deep = (deep_ok && per_cta <= deep_cap) ? 1 : 0;
        a.split_merge = (deep_ok && per_cta > deep_cap) ? 1 : 0;
      }
      // Two key chunks per (sequence, head), one round of block-row units, unpacked heads, one-plane operands:
      // the two chunks of a head run as a pair of CTAs that merge through distributed shared memory.
      if (!c->split && a.pack == 1 && a.merge_deep && !a.split_merge && !c->knobs.no_pair && c->g.block_len <= 32 &&
          units_stream == ns && (ns % 2) == 0 && (a.n_ctas % 2) == 0) {
        if (plan.pair < 0) {
          plan.pair = 1;
          for (int i = 0; i < list.n; ++i)
            if (c->items_host[list.off + i].pad != 2) plan.pair = 0;
        }
        a.pair_chunks = plan.pair;
      }
      if (c->knobs.verbose && a.pair_chunks) {
        static int printed_pair = 0;
        if (printed_pair++ < 4) fprintf(stderr, "lacache: step plan (block %d): the two key chunks of a head run as a pair of CTAs\n", blk);
      }
    } else {
      a.n_ctas_stream = (int)std::min<long long>(c->num_sms, units_stream);
      a.n_ctas = a.n_ctas_stream;
      // (a plain build writes the cached state itself: the buffer the tensor map of the state describes)
      a.st_tma = (mode == MODE_BUILD && !c->split && !c->knobs.no_staged_state) ? 1 : 0;
    }
  }
  return a;
}

// one launch of the tcgen05 kernel; with a span ring set, the launch gets the ring's next slot
cudaError_t launch_tc(lacache_ctx* c, AttnArgs a, const TcMaps* maps, cudaStream_t s) {
  if (c->span_ring) a.span = c->span_ring + 2 * (size_t)(c->span_next++ % (unsigned)c->span_slots);
  return tc_attention(c->g, a, maps, s);
}

lacache_status run_attention(lacache_ctx* c, const AttnArgs& a, bool scratch, cudaStream_t s) {
  if (c->engine == LACACHE_ENGINE_TCGEN05 && a.out) {
    if (!tc_set_out(scratch ? c->maps_scratch : c->maps, c->g, a.out, a.out_bf16 != 0, c->err, sizeof(c->err))) return LACACHE_ERR_CUDA;
  }
  if (c->ev_start) CU_TRY(c, cudaEventRecord(c->ev_start, s));
  if (c->engine == LACACHE_ENGINE_TCGEN05 && a.split_merge) {
    // The pipelined merge variant tabulates at most TC_DEEP_MAX_UNITS units per CTA.  A step with more
    // fixed rows than that goes out in several launches: the first carries the block queries and as
    // many row tiles as its merge CTAs can tabulate, the others row tiles only, on all SMs.
    const TcMaps* maps = scratch ? c->maps_scratch : c->maps;
    const int Hq = c->g.Hq;
    const int deep_cap = deep_unit_cap(c);
    AttnArgs b = a;
    b.merge_deep = 1;
    const int m0 = a.n_ctas - a.n_ctas_stream;
    int done = std::min(a.n_items_merge, std::max(1, deep_cap * m0 / Hq));
    b.n_items_merge = done;
    b.n_ctas = a.n_ctas_stream + (int)std::min<long long>((long long)done * Hq, m0);
    CU_TRY(c, launch_tc(c, b, maps, s));
    c->last_launches++;
    const int rest = a.n_items_merge - done;
    if (rest > 0) {
      const int cap = std::max(1, deep_cap * c->num_sms / Hq);
      const int n_more = (rest + cap - 1) / cap;
      const int per = (rest + n_more - 1) / n_more;
      while (done < a.n_items_merge) {
        AttnArgs m = a;
        m.merge_deep = 1;
        m.n_items = 0;
        m.n_ctas_stream = 0;
        m.items_merge = a.items_merge + done;
        m.n_items_merge = std::min(per, a.n_items_merge - done);
        m.n_ctas = (int)std::min<long long>(c->num_sms, (long long)m.n_items_merge * Hq);
        CU_TRY(c, launch_tc(c, m, maps, s));
        c->last_launches++;
        done += m.n_items_merge;
      }
    }
  } else {
    if (c->engine == LACACHE_ENGINE_TCGEN05)
      CU_TRY(c, launch_tc(c, a, scratch ? c->maps_scratch : c->maps, s));
    else
      CU_TRY(c, simt_attention(c->g, a, s));
    c->last_launches++;
  }
  if (c->ev_stop) CU_TRY(c, cudaEventRecord(c->ev_stop, s));
  return LACACHE_OK;
}

lacache_status rope_all(lacache_ctx* c, const void* q, const void* k, const void* v, const RotBuffers& dst,
                        cudaStream_t s) {
  RopeArgs r{};
  r.q = q; r.k = k; r.v = v;
  r.n_src_rows = c->g.T;
  r.blk_start = nullptr; r.block_len = c->g.block_len;
  r.pos_of_tok = c->d_pos; r.cos_tab = c->d_cos; r.sin_tab = c->d_sin;
  r.dst = dst;
  r.in_dtype = c->cfg.dtype;
  CU_TRY(c, rope_write(c->g, r, c->engine, s));
  c->last_launches++;
  return LACACHE_OK;
}

lacache_status ensure_staging(lacache_ctx* c) {
  if (c->hs_out[0]) return LACACHE_OK;
  const Geometry& g = c->g;
  size_t es = elem_size(c->cfg.dtype);
  size_t nq = (size_t)g.T * g.Hq * g.d, nk = (size_t)g.T * g.Hkv * g.d;
  size_t bq = (size_t)g.B * g.block_len * g.Hq * g.d, bk = (size_t)g.B * g.block_len * g.Hkv * g.d;
  uint8_t *a, *b, *cc, *d, *e, *f;
  CU_TRY(c, dev_alloc(c, &a, nq * es));
  CU_TRY(c, dev_alloc(c, &b, nk * es));
  CU_TRY(c, dev_alloc(c, &cc, nk * es));
  CU_TRY(c, dev_alloc(c, &d, bq * es));
  CU_TRY(c, dev_alloc(c, &e, bk * es));
  CU_TRY(c, dev_alloc(c, &f, bk * es));
  c->hs_q = a; c->hs_k = b; c->hs_v = cc; c->hs_qb = d; c->hs_kb = e; c->hs_vb = f;
  const size_t out_elems = c->cfg.out_dtype == LACACHE_OUT_BF16 ? (nq + 1) / 2 : nq;   // in floats
  for (int b = 0; b < 2; ++b) {
    CU_TRY(c, dev_alloc(c, &c->hs_lse[b], (size_t)g.T * g.Hq));
    CU_TRY(c, cudaEventCreateWithFlags(&c->ev_ready[b], cudaEventDisableTiming));
    CU_TRY(c, cudaEventCreateWithFlags(&c->ev_copied[b], cudaEventDisableTiming));
  }
  CU_TRY(c, cudaStreamCreateWithFlags(&c->copy_stream, cudaStreamNonBlocking));
  CU_TRY(c, dev_alloc(c, &c->hs_out[1], out_elems));
  CU_TRY(c, dev_alloc(c, &c->hs_out[0], out_elems));   // (last: its being set marks the staging as complete)
  return LACACHE_OK;
}

}  // namespace

namespace lacache {
// lets other translation units of the library set the text behind lacache_last_error(NULL)
void set_thread_error(const char* msg) { snprintf(g_create_err, sizeof(g_create_err), "%s", msg); }
}  // namespace lacache

extern "C" {

int lacache_version(void) { return 100; }

lacache_status lacache_create(const lacache_config* cfg, lacache_ctx** out) {
  if (out) *out = nullptr;
  g_create_err[0] = 0;
  if (!cfg || !out) return fail(nullptr, LACACHE_ERR_INVALID_ARG, "cfg or out is NULL");
  lacache_ctx* c = new (std::nothrow) lacache_ctx();
  if (!c) return fail(nullptr, LACACHE_ERR_OOM, "host allocation failed");
  lacache_status st = create_impl(cfg, c);
  if (st != LACACHE_OK) {
    snprintf(g_create_err, sizeof(g_create_err), "%s", c->err);
    cudaGetLastError();
    destroy_impl(c);
    return st;
  }
  *out = c;
  return LACACHE_OK;
}

lacache_status lacache_destroy(lacache_ctx* ctx) {
  if (!ctx) return LACACHE_ERR_INVALID_ARG;
  destroy_impl(ctx);
  return LACACHE_OK;
}

namespace {
lacache_status run_window(lacache_ctx* c, lacache_ctx::ListRef list, int blk, const StateBuffers& init,
                          const StateBuffers& dst, const StateBuffers& snap, cudaStream_t s, float* out = nullptr,
                          float* lse = nullptr);
}  // namespace

lacache_status lacache_build(lacache_ctx* c, int block_idx, const void* q, const void* k, const void* v,
                             void* stream) {
  if (!c) return LACACHE_ERR_INVALID_ARG;
  if (!q || !k || !v) return fail(c, LACACHE_ERR_INVALID_ARG, "NULL input pointer");
  if (misaligned(q) || misaligned(k) || misaligned(v)) return fail(c, LACACHE_ERR_INVALID_ARG, "input pointer not 16-byte aligned");
  if (block_idx < 0 || block_idx >= c->g.n_blk)
    return fail(c, LACACHE_ERR_INVALID_ARG, "block_idx %d outside [0, %d)", block_idx, c->g.n_blk);
  cudaStream_t s = (cudaStream_t)stream;
  c->last_launches = 0;
  c->built_block = -1;
  c->prefix_block = -1;
  lacache_status st = rope_all(c, q, k, v, c->rot, s);
  if (st != LACACHE_OK) return st;
  if (c->cfg.cache_granularity == LACACHE_GRANULARITY_TILE) {
    // state of the rows outside the tiles that overlap the block: over the key tiles before them, then
    // continued over the key tiles after them (in place: a unit loads its rows before it stores them)
    st = run_window(c, c->tile_prefix[block_idx], block_idx, StateBuffers{}, c->st, StateBuffers{}, s);
    if (st != LACACHE_OK) return st;
    st = run_window(c, c->tile_suffix[block_idx], block_idx, c->st, c->st, StateBuffers{}, s);
    if (st != LACACHE_OK) return st;
  } else {
    AttnArgs a = attn_args(c, MODE_BUILD, c->build_list[block_idx], block_idx, c->rot, nullptr, nullptr);
    st = run_attention(c, a, false, s);
    if (st != LACACHE_OK) return st;
  }
  c->built_block = block_idx;
  c->steps_since_build = 0;
  return LACACHE_OK;
}

namespace {
// the prefix state's buffers, allocated when the incremental build is first used
lacache_status ensure_prefix_state(lacache_ctx* c) {
  if (c->engine != LACACHE_ENGINE_TCGEN05)
    return fail(c, LACACHE_ERR_UNSUPPORTED, "the incremental build needs the tcgen05 engine");
  if (c->cfg.cache_granularity == LACACHE_GRANULARITY_TILE)
    return fail(c, LACACHE_ERR_UNSUPPORTED, "the incremental build is token-granular only");
  if (c->pst.o) return LACACHE_OK;
  const Geometry& g = c->g;
  CU_TRY(c, dev_alloc(c, &c->pst.m, (size_t)g.Hq * g.Tp, true));
  CU_TRY(c, dev_alloc(c, &c->pst.l, (size_t)g.Hq * g.Tp, true));
  CU_TRY(c, dev_alloc(c, &c->pst.o, (size_t)g.Hq * g.Tp * g.d, true));
  return LACACHE_OK;
}
// one launch over a list of key-window items: dst = (init +) the window's keys
// Block-row units of the step kernel (key chunks, heads of a KV group packed) whose merged result is the
// rows' state, stored to dst, instead of normalised rows; no fixed-row units, nothing rotated on the fly.
lacache_status run_block_rows_to_state(lacache_ctx* c, lacache_ctx::ListRef list, int blk, const StateBuffers& dst,
                                       cudaStream_t s) {
  if (list.n == 0) return LACACHE_OK;
  AttnArgs a = attn_args(c, MODE_FULL, list, blk, c->rot, nullptr, nullptr);
  a.mode = MODE_STEP;
  set_packing(c, a);
  a.n_ctas_stream = (int)std::min<long long>(c->num_sms, (long long)list.n * a.stream_slots);
  a.n_ctas = a.n_ctas_stream;
  a.blk_to_state = 1;   // the units leave partial states ...
  lacache_status st = run_attention(c, a, false, s);
  if (st != LACACHE_OK) return st;
  ChunkMergeArgs m{};    // ... which a launch over all rows and heads merges (the last chunk to arrive, as in a
                         // step, would merge its heads alone, one L2 round trip after the other)
  m.part_m = c->part_m; m.part_l = c->part_l; m.part_o = c->part_o;
  m.max_chunks = c->part_chunks;
  m.tab = c->d_adv_tab + (size_t)blk * c->g.B * 2;
  m.st = dst;
  m.no_pdl = c->knobs.no_pdl ? 1 : 0;
  CU_TRY(c, merge_chunk_states(c->g, m, s));
  c->last_launches++;
  return LACACHE_OK;
}

lacache_status run_window(lacache_ctx* c, lacache_ctx::ListRef list, int blk, const StateBuffers& init,
                          const StateBuffers& dst, const StateBuffers& snap, cudaStream_t s, float* out, float* lse) {
  if (list.n == 0) return LACACHE_OK;
  AttnArgs a = attn_args(c, MODE_BUILD, list, blk, c->rot, out, lse);
  a.window = 1;
  a.init = init;
  a.st = dst;
  a.snap = snap;
  return run_attention(c, a, false, s);
}
}  // namespace

lacache_status lacache_build_incremental(lacache_ctx* c, int block_idx, const void* q, const void* k, const void* v,
                                         void* stream) {
  if (!c) return LACACHE_ERR_INVALID_ARG;
  if (!q || !k || !v) return fail(c, LACACHE_ERR_INVALID_ARG, "NULL input pointer");
  if (misaligned(q) || misaligned(k) || misaligned(v)) return fail(c, LACACHE_ERR_INVALID_ARG, "input pointer not 16-byte aligned");
  if (block_idx < 0 || block_idx >= c->g.n_blk)
    return fail(c, LACACHE_ERR_INVALID_ARG, "block_idx %d outside [0, %d)", block_idx, c->g.n_blk);
  lacache_status st = ensure_prefix_state(c);
  if (st != LACACHE_OK) return st;
  cudaStream_t s = (cudaStream_t)stream;
  c->last_launches = 0;
  c->built_block = -1;
  c->prefix_block = -1;
  st = rope_all(c, q, k, v, c->rot, s);
  if (st != LACACHE_OK) return st;
  st = run_window(c, c->inc_prefix[block_idx], block_idx, StateBuffers{}, c->pst, StateBuffers{}, s);
  if (st != LACACHE_OK) return st;
  st = run_window(c, c->inc_comb[block_idx], block_idx, c->pst, c->st, StateBuffers{}, s);
  if (st != LACACHE_OK) return st;
  c->built_block = block_idx;
  c->prefix_block = block_idx;
  c->steps_since_build = 0;
  return LACACHE_OK;
}

lacache_status lacache_build_advance(lacache_ctx* c, const void* q, const void* k, const void* v, void* stream) {
  if (!c) return LACACHE_ERR_INVALID_ARG;
  if (c->built_block < 0 || c->prefix_block != c->built_block)
    return fail(c, LACACHE_ERR_STATE, "lacache_build_advance needs the state of lacache_build_incremental or of an earlier advance");
  if (c->built_block + 1 >= c->g.n_blk)
    return fail(c, LACACHE_ERR_STATE, "block %d is the last one", c->built_block);
  if (!q || !k || !v) return fail(c, LACACHE_ERR_INVALID_ARG, "NULL input pointer");
  if (misaligned(q) || misaligned(k) || misaligned(v)) return fail(c, LACACHE_ERR_INVALID_ARG, "input pointer not 16-byte aligned");
  cudaStream_t s = (cudaStream_t)stream;
  const int done = c->built_block, blk = done + 1;
  c->last_launches = 0;
  c->built_block = -1;
  c->prefix_block = -1;
  // the finished block's rows, rotated into the cache (an ordinary launch: everything ahead in the
  // stream, a step that still reads the cached state included, completes first)
  RopeArgs r{};
  r.q = q; r.k = k; r.v = v;
  r.n_src_rows = c->g.B * c->g.block_len;
  r.blk_start = c->d_blk_start_all + (size_t)done * c->g.B;
  r.block_len = c->g.block_len;
  r.pos_of_tok = c->d_pos; r.cos_tab = c->d_cos; r.sin_tab = c->d_sin;
  {
    const size_t row0 = (size_t)done * c->g.B * c->g.block_len;
    r.row_tok = c->d_blk_tok + row0;
    r.row_cos = c->d_blk_cos + row0 * (c->g.d / 2);
    r.row_sin = c->d_blk_sin + row0 * (c->g.d / 2);
  }
  r.pdl = 0;
  r.dst = c->rot;
  r.in_dtype = c->cfg.dtype;
  CU_TRY(c, rope_write(c->g, r, c->engine, s));
  c->last_launches++;
  lacache_status st = c->knobs.no_chunked_advance ? run_window(c, c->inc_fresh[blk], blk, StateBuffers{}, c->pst, StateBuffers{}, s)
                                                  : run_block_rows_to_state(c, c->inc_fresh_chunks[blk], blk, c->pst, s);
  if (st != LACACHE_OK) return st;
  if (c->knobs.verbose) {   // which of the two launches a device status belongs to
    int32_t hs[4] = {0, 0, 0, 0};
    cudaStreamSynchronize(s);
    cudaMemcpy(hs, c->d_status, sizeof(hs), cudaMemcpyDeviceToHost);
    fprintf(stderr, "lacache: advance to block %d, after the finished block's rows: status %d %d %d %d\n", blk, hs[0], hs[1], hs[2], hs[3]);
  }
  st = run_window(c, c->inc_fused[blk], blk, c->pst, c->st, c->pst, s);
  if (st != LACACHE_OK) return st;
  c->built_block = blk;
  c->prefix_block = blk;
  c->steps_since_build = 0;
  return LACACHE_OK;
}

namespace {
// inputs_just_written: q / k / v are produced by the kernel enqueued right before this call, so
// nothing of the step may read them before that kernel has completed
lacache_status step_impl(lacache_ctx* c, const void* q, const void* k, const void* v, float* out, float* lse,
                         void* stream, bool inputs_just_written);
}  // namespace

lacache_status lacache_step(lacache_ctx* c, const void* q, const void* k, const void* v, float* out,
                            float* lse, void* stream) {
  return step_impl(c, q, k, v, out, lse, stream, false);
}

namespace {
// the producer handle fits the context and covers n tokens
lacache_status check_producer(lacache_ctx* c, lacache_qkv* p, int n) {
  int hq = 0, hkv = 0, max_tokens = 0;
  const int d = qkv_heads(p, &hq, &hkv, &max_tokens);
  if (c->cfg.dtype != LACACHE_DTYPE_BF16) return fail(c, LACACHE_ERR_UNSUPPORTED, "the producer writes bf16: the context must be bf16");
  if (hq != c->g.Hq || hkv != c->g.Hkv || d != c->g.d)
    return fail(c, LACACHE_ERR_SHAPE, "producer heads %d/%d x %d, context %d/%d x %d", hq, hkv, d, c->g.Hq, c->g.Hkv, c->g.d);
  if (n > max_tokens) return fail(c, LACACHE_ERR_SHAPE, "%d tokens, producer max_tokens %d", n, max_tokens);
  return LACACHE_OK;
}
}  // namespace

lacache_status lacache_build_tokens(lacache_ctx* c, lacache_qkv* p, int block_idx, const int32_t* token_ids,
                                    const void* hidden, void* stream) {
  if (!c || !p) return LACACHE_ERR_INVALID_ARG;
  lacache_status st = check_producer(c, p, c->g.T);
  if (st != LACACHE_OK) return st;
  void *q, *k, *v;
  qkv_scratch(p, false, &q, &k, &v);
  qkv_set_full_owner(p, nullptr, 0);
  st = lacache_qkv_project(p, token_ids, hidden, c->g.T, q, k, v, nullptr, stream);
  if (st != LACACHE_OK) return fail(c, st, "producer: %s", lacache_qkv_last_error(p));
  st = lacache_build(c, block_idx, q, k, v, stream);
  if (st != LACACHE_OK) return st;
  qkv_set_full_owner(p, c, c->g.T);
  c->last_launches += lacache_qkv_last_launch_count(p);
  return LACACHE_OK;
}

lacache_status lacache_build_tokens_update(lacache_ctx* c, lacache_qkv* p, int block_idx, const int32_t* rows,
                                           const int32_t* token_ids, const void* hidden, int n_changed,
                                           void* stream) {
  if (!c || !p) return LACACHE_ERR_INVALID_ARG;
  if (n_changed < 0 || n_changed > c->g.T) return fail(c, LACACHE_ERR_SHAPE, "n_changed %d outside [0, %d]", n_changed, c->g.T);
  lacache_status st = check_producer(c, p, c->g.T);
  if (st != LACACHE_OK) return st;
  if (!qkv_full_owner_is(p, c, c->g.T))
    return fail(c, LACACHE_ERR_STATE, "lacache_build_tokens_update needs a preceding lacache_build_tokens of this context with this producer");
  if (n_changed > 0 && !rows) return fail(c, LACACHE_ERR_INVALID_ARG, "NULL rows");
  void *q, *k, *v;
  qkv_scratch(p, false, &q, &k, &v);
  int producer_launches = 0;
  if (n_changed > 0) {
    st = qkv_project_rows(p, token_ids, hidden, n_changed, q, k, v, nullptr, rows, c->g.T, false, stream);
    if (st != LACACHE_OK) return fail(c, st, "producer: %s", lacache_qkv_last_error(p));
    producer_launches = lacache_qkv_last_launch_count(p);
  }
  st = lacache_build(c, block_idx, q, k, v, stream);
  if (st == LACACHE_OK) c->last_launches += producer_launches;
  return st;
}

lacache_status lacache_build_tokens_incremental(lacache_ctx* c, lacache_qkv* p, int block_idx,
                                                const int32_t* token_ids, const void* hidden, void* stream) {
  if (!c || !p) return LACACHE_ERR_INVALID_ARG;
  lacache_status st = check_producer(c, p, c->g.T);
  if (st != LACACHE_OK) return st;
  void *q, *k, *v;
  qkv_scratch(p, false, &q, &k, &v);
  qkv_set_full_owner(p, nullptr, 0);
  st = lacache_qkv_project(p, token_ids, hidden, c->g.T, q, k, v, nullptr, stream);
  if (st != LACACHE_OK) return fail(c, st, "producer: %s", lacache_qkv_last_error(p));
  st = lacache_build_incremental(c, block_idx, q, k, v, stream);
  if (st == LACACHE_OK) c->last_launches += lacache_qkv_last_launch_count(p);
  return st;
}

lacache_status lacache_build_advance_tokens(lacache_ctx* c, lacache_qkv* p, const int32_t* fin_token_ids,
                                            const void* fin_hidden, void* stream) {
  if (!c || !p) return LACACHE_ERR_INVALID_ARG;
  if (c->built_block < 0 || c->prefix_block != c->built_block)
    return fail(c, LACACHE_ERR_STATE, "lacache_build_advance_tokens needs the state of an incremental build or of an earlier advance");
  const int n = c->g.B * c->g.block_len;
  lacache_status st = check_producer(c, p, n);
  if (st != LACACHE_OK) return st;
  void *q, *k, *v;
  qkv_scratch(p, true, &q, &k, &v);
  // (the RoPE launch of the advance is an ordinary one: it starts when the projection has completed)
  st = qkv_project_rows(p, fin_token_ids, fin_hidden, n, q, k, v, nullptr, nullptr, 0, false, stream);
  if (st != LACACHE_OK) return fail(c, st, "producer: %s", lacache_qkv_last_error(p));
  st = lacache_build_advance(c, q, k, v, stream);
  if (st == LACACHE_OK) c->last_launches += lacache_qkv_last_launch_count(p);
  return st;
}

lacache_status lacache_step_tokens(lacache_ctx* c, lacache_qkv* p, const int32_t* blk_token_ids,
                                   const void* blk_hidden, float* out, float* lse, void* stream) {
  if (!c || !p) return LACACHE_ERR_INVALID_ARG;
  if (c->built_block < 0) return fail(c, LACACHE_ERR_STATE, "lacache_step_tokens before a successful build");
  const int n = c->g.B * c->g.block_len;
  lacache_status st = check_producer(c, p, n);
  if (st != LACACHE_OK) return st;
  void *q, *k, *v;
  qkv_scratch(p, true, &q, &k, &v);
  // with the cross-step overlap on (and not right after a build) the norm kernel reads the ids while the
  // previous step's attention kernel still runs: the same contract as for q_blk / k_blk / v_blk of lacache_step
  const bool early = c->step_overlap && c->steps_since_build > 0 && !c->knobs.no_pdl && !c->knobs.no_step_overlap;
  st = qkv_project_rows(p, blk_token_ids, blk_hidden, n, q, k, v, nullptr, nullptr, 0, early, stream);
  if (st != LACACHE_OK) return fail(c, st, "producer: %s", lacache_qkv_last_error(p));
  st = step_impl(c, q, k, v, out, lse, stream, true);
  if (st == LACACHE_OK) c->last_launches += lacache_qkv_last_launch_count(p);
  return st;
}

namespace {
lacache_status step_impl(lacache_ctx* c, const void* q, const void* k, const void* v, float* out, float* lse,
                         void* stream, bool inputs_just_written) {
  if (!c) return LACACHE_ERR_INVALID_ARG;
  if (c->built_block < 0) return fail(c, LACACHE_ERR_STATE, "lacache_step before a successful lacache_build");
  if (!q || !k || !v || !out) return fail(c, LACACHE_ERR_INVALID_ARG, "NULL pointer");
  if (misaligned(q) || misaligned(k) || misaligned(v) || misaligned(out) || (lse && misaligned(lse)))
    return fail(c, LACACHE_ERR_INVALID_ARG, "pointer not 16-byte aligned");
  cudaStream_t s = (cudaStream_t)stream;
  const int blk = c->built_block;
  c->last_launches = 0;
  RopeArgs r{};
  r.q = q; r.k = k; r.v = v;
  r.n_src_rows = c->g.B * c->g.block_len;
  r.blk_start = c->d_blk_start_all + (size_t)blk * c->g.B;
  r.block_len = c->g.block_len;
  r.pos_of_tok = c->d_pos; r.cos_tab = c->d_cos; r.sin_tab = c->d_sin;
  {
    const size_t row0 = (size_t)blk * c->g.B * c->g.block_len;
    r.row_tok = c->d_blk_tok + row0;
    r.row_cos = c->d_blk_cos + row0 * (c->g.d / 2);
    r.row_sin = c->d_blk_sin + row0 * (c->g.d / 2);
  }
  // may start while the previous step's attention kernel drains (it waits before its stores); when
  // the kernel before it in the stream is the one that writes its inputs, it waits for that one first
  const bool overlap = c->step_overlap && !c->knobs.no_pdl && !c->knobs.no_step_overlap;
  // (the first step after a build is launched the ordinary way: the build's cached state, which the
  // attention kernel reads before it waits on anything, is then complete and flushed)
  r.pdl = inputs_just_written ? 2 : ((overlap && c->steps_since_build > 0) ? 1 : 0);
  r.no_pdl = (c->knobs.no_pdl || c->knobs.no_step_overlap) ? 1 : 0;
  c->steps_since_build++;
  r.dst = c->rot;
  r.in_dtype = c->cfg.dtype;
  if (c->cfg.cache_granularity == LACACHE_GRANULARITY_TILE) {
    // Algorithm 1's reuse pass at tile granularity: ordinary launches, one pass of the build kernel over
    // key windows (rows of the overlapping tiles x all keys; every other row: cached state + the keys of
    // the overlapping tiles), normalised output instead of state
    r.pdl = 0;
    CU_TRY(c, rope_write(c->g, r, c->engine, s));
    c->last_launches++;
    return run_window(c, c->tile_step[blk], blk, c->st, c->st, StateBuffers{}, s, out, lse);
  }
  CU_TRY(c, rope_write(c->g, r, c->engine, s));
  c->last_launches++;
  AttnArgs a = attn_args(c, MODE_STEP, c->step_list[blk], blk, c->rot, out, lse);
  a.step_overlap = overlap ? 1 : 0;
  if (!c->knobs.no_qcomp) {
    a.q_raw = q;
    a.k_raw = k;
    a.v_raw = v;
    a.row_cos = r.row_cos;
    a.row_sin = r.row_sin;
  }
  return run_attention(c, a, false, s);
}
}  // namespace

lacache_status lacache_sample_block(lacache_ctx* c, const void* logits, int dtype, int vocab, float* conf,
                                    int32_t* token, float* lse, void* stream) {
  if (!c) return LACACHE_ERR_INVALID_ARG;
  if (c->built_block < 0) return fail(c, LACACHE_ERR_STATE, "lacache_sample_block before a successful build");
  if (!logits || !conf || !token) return fail(c, LACACHE_ERR_INVALID_ARG, "NULL pointer");
  if (dtype != LACACHE_DTYPE_BF16 && dtype != LACACHE_DTYPE_FP32) return fail(c, LACACHE_ERR_INVALID_ARG, "dtype %d", dtype);
  if (vocab <= 0) return fail(c, LACACHE_ERR_INVALID_ARG, "vocab %d", vocab);
  constexpr int MAX_SPLITS = 64;
  const int n = c->g.B * c->g.block_len;
  if (n > 65535) return fail(c, LACACHE_ERR_UNSUPPORTED, "%d block rows: the sampler's grid takes at most 65535", n);
  if (!c->sample_part) {
    CU_TRY(c, dev_alloc(c, &c->sample_part, (size_t)n * MAX_SPLITS * 4));
    CU_TRY(c, dev_alloc(c, &c->sample_counters, (size_t)n, true));
  }
  SampleArgs a{};
  a.logits = logits; a.dtype = dtype;
  a.n_tokens = c->g.T; a.vocab = vocab;
  a.rows = c->d_blk_tok + (size_t)c->built_block * n;
  a.n_rows = n;
  // as many CTAs as are resident at once (four per SM), each with at least 2048 entries, slices a
  // multiple of 8 entries (rounded down: no second wave of a few stragglers)
  int splits = std::max(1, std::min(MAX_SPLITS, 4 * c->num_sms / n));
  splits = std::min(splits, std::max(1, vocab / 2048));
  int slice = ((vocab + splits - 1) / splits + 7) / 8 * 8;
  splits = (vocab + slice - 1) / slice;
  a.splits = splits; a.slice = slice;
  const size_t row_bytes = (size_t)vocab * elem_size(dtype);
  a.vector_ok = (row_bytes % 16 == 0 && !misaligned(logits)) ? 1 : 0;
  a.part = c->sample_part; a.counters = c->sample_counters;
  a.conf = conf; a.token = token; a.lse = lse;
  a.status = c->d_status;
  c->last_launches = 0;
  CU_TRY(c, sample_rows(a, (cudaStream_t)stream));
  c->last_launches++;
  return LACACHE_OK;
}

lacache_status lacache_set_step_overlap(lacache_ctx* c, int enable) {
  if (!c) return LACACHE_ERR_INVALID_ARG;
  c->step_overlap = enable ? 1 : 0;
  return LACACHE_OK;
}

lacache_status lacache_full_recompute(lacache_ctx* c, const void* q, const void* k, const void* v, float* out,
                                      float* lse, void* stream) {
  if (!c) return LACACHE_ERR_INVALID_ARG;
  if (!q || !k || !v || !out) return fail(c, LACACHE_ERR_INVALID_ARG, "NULL pointer");
  if (misaligned(q) || misaligned(k) || misaligned(v) || misaligned(out) || (lse && misaligned(lse)))
    return fail(c, LACACHE_ERR_INVALID_ARG, "pointer not 16-byte aligned");
  cudaStream_t s = (cudaStream_t)stream;
  c->last_launches = 0;
  lacache_status st = rope_all(c, q, k, v, c->rot_scratch, s);
  if (st != LACACHE_OK) return st;
  AttnArgs a = attn_args(c, MODE_FULL, c->full_list, -1, c->rot_scratch, out, lse);
  return run_attention(c, a, true, s);
}

lacache_status lacache_build_host(lacache_ctx* c, int block_idx, const void* q, const void* k, const void* v,
                                  void* stream) {
  if (!c) return LACACHE_ERR_INVALID_ARG;
  if (!q || !k || !v) return fail(c, LACACHE_ERR_INVALID_ARG, "NULL input pointer");
  lacache_status st = ensure_staging(c);
  if (st != LACACHE_OK) return st;
  cudaStream_t s = (cudaStream_t)stream;
  const Geometry& g = c->g;
  size_t es = elem_size(c->cfg.dtype);
  CU_TRY(c, cudaMemcpyAsync(c->hs_q, q, (size_t)g.T * g.Hq * g.d * es, cudaMemcpyHostToDevice, s));
  CU_TRY(c, cudaMemcpyAsync(c->hs_k, k, (size_t)g.T * g.Hkv * g.d * es, cudaMemcpyHostToDevice, s));
  CU_TRY(c, cudaMemcpyAsync(c->hs_v, v, (size_t)g.T * g.Hkv * g.d * es, cudaMemcpyHostToDevice, s));
  return lacache_build(c, block_idx, c->hs_q, c->hs_k, c->hs_v, stream);
}

lacache_status lacache_step_host(lacache_ctx* c, const void* q, const void* k, const void* v, float* out,
                                 float* lse, void* stream) {
  if (!c) return LACACHE_ERR_INVALID_ARG;
  if (!q || !k || !v || !out) return fail(c, LACACHE_ERR_INVALID_ARG, "NULL pointer");
  lacache_status st = ensure_staging(c);
  if (st != LACACHE_OK) return st;
  cudaStream_t s = (cudaStream_t)stream;
  const Geometry& g = c->g;
  size_t es = elem_size(c->cfg.dtype);
  size_t rows = (size_t)g.B * g.block_len;
  const unsigned i = c->host_steps;
  const int b = (int)(i & 1u);
  CU_TRY(c, cudaMemcpyAsync(c->hs_qb, q, rows * g.Hq * g.d * es, cudaMemcpyHostToDevice, s));
  CU_TRY(c, cudaMemcpyAsync(c->hs_kb, k, rows * g.Hkv * g.d * es, cudaMemcpyHostToDevice, s));
  CU_TRY(c, cudaMemcpyAsync(c->hs_vb, v, rows * g.Hkv * g.d * es, cudaMemcpyHostToDevice, s));
  // the step writes the result buffer that the copy of the call before last has left
  if (i >= 2) CU_TRY(c, cudaStreamWaitEvent(s, c->ev_copied[b], 0));
  st = lacache_step(c, c->hs_qb, c->hs_kb, c->hs_vb, c->hs_out[b], lse ? c->hs_lse[b] : nullptr, stream);
  if (st != LACACHE_OK) return st;
  // ... and its copy to the host runs on the context's copy stream, beside whatever the caller's stream does
  // next (the following step, as a rule)
  CU_TRY(c, cudaEventRecord(c->ev_ready[b], s));
  CU_TRY(c, cudaStreamWaitEvent(c->copy_stream, c->ev_ready[b], 0));
  const size_t out_es = c->cfg.out_dtype == LACACHE_OUT_BF16 ? 2 : 4;
  CU_TRY(c, cudaMemcpyAsync(out, c->hs_out[b], out_es * g.T * g.Hq * g.d, cudaMemcpyDeviceToHost, c->copy_stream));
  if (lse) CU_TRY(c, cudaMemcpyAsync(lse, c->hs_lse[b], sizeof(float) * g.T * g.Hq, cudaMemcpyDeviceToHost, c->copy_stream));
  CU_TRY(c, cudaEventRecord(c->ev_copied[b], c->copy_stream));
  c->host_steps = i + 1;
  // the previous call's copy joins the caller's stream behind this call's kernels
  if (i >= 1) CU_TRY(c, cudaStreamWaitEvent(s, c->ev_copied[b ^ 1], 0));
  return LACACHE_OK;
}

lacache_status lacache_join_host(lacache_ctx* c, void* stream) {
  if (!c) return LACACHE_ERR_INVALID_ARG;
  if (c->host_steps == 0) return LACACHE_OK;
  CU_TRY(c, cudaStreamWaitEvent((cudaStream_t)stream, c->ev_copied[(c->host_steps - 1) & 1u], 0));
  return LACACHE_OK;
}

lacache_status lacache_export_state(lacache_ctx* c, float* m, float* l, float* o, void* stream) {
  if (!c) return LACACHE_ERR_INVALID_ARG;
  if (c->built_block < 0) return fail(c, LACACHE_ERR_STATE, "no state: lacache_build has not run");
  ExportArgs e{};
  e.rot = c->rot; e.st = c->st; e.m = m; e.l = l; e.o = o;
  CU_TRY(c, export_buffers(c->g, e, c->engine, (cudaStream_t)stream));
  return LACACHE_OK;
}

lacache_status lacache_export_rope_cache(lacache_ctx* c, float* q, float* k, float* v, void* stream) {
  if (!c) return LACACHE_ERR_INVALID_ARG;
  ExportArgs e{};
  e.rot = c->rot; e.st = c->st; e.q_rot = q; e.k_rot = k; e.v = v;
  CU_TRY(c, export_buffers(c->g, e, c->engine, (cudaStream_t)stream));
  return LACACHE_OK;
}

lacache_status lacache_export_index_meta(lacache_ctx* c, int32_t* seq, int32_t* pos, int32_t* isb, int32_t* kvh) {
  if (!c) return LACACHE_ERR_INVALID_ARG;
  const Geometry& g = c->g;
  if (seq) memcpy(seq, c->seq_of_tok.data(), sizeof(int32_t) * g.T);
  if (pos) memcpy(pos, c->pos_of_tok.data(), sizeof(int32_t) * g.T);
  if (isb) {
    memset(isb, 0, sizeof(int32_t) * g.T);
    if (c->built_block >= 0)
      for (int b = 0; b < g.B; ++b) {
        int bs = c->blk_start_all[(size_t)c->built_block * g.B + b];
        for (int r = 0; r < g.block_len; ++r) isb[bs + r] = 1;
      }
  }
  if (kvh)
    for (int h = 0; h < g.Hq; ++h) kvh[h] = h / g.group;
  return LACACHE_OK;
}

lacache_status lacache_set_span_ring(lacache_ctx* c, uint64_t* ring, int n_slots) {
  if (!c) return LACACHE_ERR_INVALID_ARG;
  if ((ring == nullptr) != (n_slots <= 0)) return fail(c, LACACHE_ERR_INVALID_ARG, "pass a ring with n_slots > 0, or NULL with 0");
  if (ring && (reinterpret_cast<uintptr_t>(ring) & 7u)) return fail(c, LACACHE_ERR_INVALID_ARG, "ring not 8-byte aligned");
  c->span_ring = reinterpret_cast<unsigned long long*>(ring);
  c->span_slots = ring ? n_slots : 0;
  c->span_next = 0;
  return LACACHE_OK;
}

lacache_status lacache_set_timing_events(lacache_ctx* c, void* ev_start, void* ev_stop) {
  if (!c) return LACACHE_ERR_INVALID_ARG;
  if ((ev_start == nullptr) != (ev_stop == nullptr)) return fail(c, LACACHE_ERR_INVALID_ARG, "pass both events or neither");
  c->ev_start = (cudaEvent_t)ev_start;
  c->ev_stop = (cudaEvent_t)ev_stop;
  return LACACHE_OK;
}

int lacache_total_tokens(const lacache_ctx* c) { return c ? c->g.T : -1; }
int lacache_last_launch_count(const lacache_ctx* c) { return c ? c->last_launches : -1; }
int lacache_engine(const lacache_ctx* c) { return c ? c->engine : -1; }

lacache_status lacache_poll_status(lacache_ctx* c) {
  if (!c) return LACACHE_ERR_INVALID_ARG;
  CU_TRY(c, cudaDeviceSynchronize());
  int32_t w[4];
  CU_TRY(c, cudaMemcpy(w, c->d_status, sizeof(w), cudaMemcpyDeviceToHost));
  if (w[0] != 0) {
    fail(c, (lacache_status)w[0], "device status: code %d at location %d (aux %d, %d)", w[0], w[1], w[2], w[3]);
    cudaMemset(c->d_status, 0, sizeof(w));
    return (lacache_status)w[0];
  }
  return LACACHE_OK;
}

const char* lacache_last_error(const lacache_ctx* c) { return c ? c->err : g_create_err; }

}  // extern "C"
