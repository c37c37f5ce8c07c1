// Internal declarations shared by the host side (lacache_api.cu) and the two
// kernel families (lacache_simt.cu: CUDA-core fp32; lacache_tc.cu: tcgen05).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/lacache.h"

namespace lacache {

// Work item kinds.  A launch walks a list of items; blockIdx.y is the q head.
enum ItemKind : int32_t {
  ITEM_ROWS = 0,   // a tile of query rows [row0, row0 + nrows) of one sequence
  ITEM_BLOCK_CHUNK = 1,  // the block's query rows x one chunk of key tiles
  ITEM_ROWS_WINDOW = 2,  // (build) a tile of query rows x the keys [kt0, kt1) of its sequence, given as token
                         // indices; key tiles are counted from token `pad` (<= kt0, may be negative).
                         // chunk bit 0: continue from the rows' state in AttnArgs::init; bit 1: store the
                         // state after the first key tile to AttnArgs::snap; bit 2: leave out the keys of
                         // the block at blk_start; bit 3: the first tile ends at blk_start (pad = blk_start -
                         // tile width) and the tiles after it are counted from the end of that block; bit 4:
                         // the unit writes normalised rows to out / lse instead of a state
};
struct WorkItem {
  int32_t kind;   // ItemKind
  int32_t seq;    // sequence index
  int32_t row0;   // first packed token index of the query rows
  int32_t nrows;  // number of valid query rows (<= tile rows)
  int32_t chunk;  // ITEM_BLOCK_CHUNK: chunk index; else 0
  int32_t kt0;    // ITEM_BLOCK_CHUNK: first key tile of the chunk
  int32_t kt1;    // ITEM_BLOCK_CHUNK: one past the last key tile
  int32_t pad;    // ITEM_BLOCK_CHUNK: number of chunks of this (sequence, block)
  int32_t seq_start;  // first packed token of the sequence
  int32_t seq_end;    // one past its last token
  int32_t blk_start;  // first packed token of the sequence's current block
  int32_t pad2;
};

// What a launch computes for ITEM_ROWS items.
enum Mode : int32_t {
  MODE_BUILD = 0,   // fixed queries x fixed keys -> cached state
  MODE_STEP = 1,    // ITEM_ROWS: fixed queries x block keys merged into the
                    // cached state; ITEM_BLOCK_CHUNK: block queries x all keys
  MODE_FULL = 2,    // every query x every key, no cache
};

// Device status word layout (int32 x 4): [0] code, [1] location, [2], [3] aux
enum StatusLoc : int32_t {
  LOC_NONE = 0,
  LOC_SMEM_ALIGN = 1,
  LOC_WAIT_Q = 2,
  LOC_WAIT_K = 3,
  LOC_WAIT_V = 4,
  LOC_WAIT_S = 5,
  LOC_WAIT_O = 6,
  LOC_UNIT_TABLE = 7,
  LOC_SAMPLE_ROW = 8,
};

struct Geometry {
  int B, T, Tp, maxN;
  int Hq, Hkv, d, group;
  int gen_len, block_len, n_blk;
  float scale_log2;  // softmax_scale * log2(e)
  int op_f16;        // tcgen05 engine, one-plane modes: the rotated Q', K' planes hold fp16 (else bf16)
};

// Rotated cache / scratch set.  SIMT engine: fp32 planes (q, k, v).
// tcgen05 engine: bf16 hi/lo planes for q and k, fp16 plane for v.
// All planes are head-major: [H][Tp][d].
struct RotBuffers {
  void* q_hi; void* q_lo;   // SIMT: q_hi = fp32 q, q_lo unused
  void* k_hi; void* k_lo;
  void* v;
};

struct StateBuffers {       // head-major: m,l [Hq][Tp]; o [Hq][Tp][d]
  float* m; float* l; float* o;   // m in log2 units (reference exponent)
};

struct RopeArgs {
  const void* q; const void* k; const void* v;  // source rows, token-major
  int n_src_rows;
  // destination token of source row r: dst_map == nullptr ? r
  //   : blk_start[r / block_len] + r % block_len
  const int32_t* blk_start; int block_len;
  const int32_t* pos_of_tok;
  const float* cos_tab; const float* sin_tab;  // [maxN][d/2]
  // optional (block rows of a step): destination token and cos/sin rows of source
  // row r, gathered ahead of time so that no load of the kernel depends on another
  const int32_t* row_tok; const float* row_cos; const float* row_sin;  // [n_src_rows], [n_src_rows][d/2]
  RotBuffers dst;
  int in_dtype;
  // launch programmatically dependent on the kernel before it in the stream.  1: that kernel is a
  // step's attention kernel, which lets its successors start early; this kernel then waits before its
  // first store.  2: that kernel writes this kernel's inputs; this kernel waits before anything else.
  int pdl;
  int no_pdl;   // host only: launch the ordinary way whatever `pdl` says (experiment knob)
};

struct AttnArgs {
  int mode;
  const WorkItem* items; int n_items;   // SIMT: all items; tcgen05: stream-role items
  // tcgen05 only: items of the merge role (fixed rows of a step), CTA split
  const WorkItem* items_merge; int n_items_merge;
  int n_ctas_stream; int n_ctas;
  // tcgen05, stream role: units per item.  Normally one per query head.  In a step of a GQA model the
  // block rows of `pack` query heads of one KV group share a 128-row tile (they read the same keys and
  // values): units then count (KV head, group of `pack` heads) pairs, each head taking `pack_rows` lanes.
  int stream_slots; int pack; int pack_rows;
  int merge_deep;            // merge role runs its pipelined variant (block_len <= 32, bounded units per CTA)
  int split_merge;           // host only: more merge units per CTA than the pipelined variant tabulates, so the
                             // fixed rows of the step go out in several launches of that variant
  // step only: the block's pre-RoPE queries [B * block_len, Hq, d] and the cos/sin rows of
  // those tokens [B * block_len][d/2]; a CTA's first block-query unit rotates its Q tile
  // from these itself and so does not have to wait for the RoPE kernel
  const void* q_raw; const float* row_cos; const float* row_sin;   // (bf16: the tcgen05 engine takes bf16 inputs only)
  // likewise the block's pre-RoPE keys and values [B * block_len, Hkv, d]: the first unit of a
  // pipelined merge-role CTA rotates the block's keys / converts its values itself
  const void* k_raw; const void* v_raw;
  int step_overlap;          // step: let the next step's kernels be scheduled while this one drains
  const int32_t* cu;         // [B+1]
  const int32_t* blk_start;  // [B] absolute token index of the block's first row
  RotBuffers rot;
  StateBuffers st;
  int window;                // build: the items are ITEM_ROWS_WINDOW (the kernel instantiation that knows them)
  StateBuffers init;         // build over key windows: the state units with the init bit start from (may alias st)
  StateBuffers snap;         // ... and where units with the snapshot bit store their state after the first key tile
                             // (may alias init: a unit loads its rows before it stores them)
  float* out; float* lse;    // token-major [T,Hq,d], [T,Hq]
  int out_bf16;              // `out` holds bf16 elements (lse stays fp32)
  // split-key partial states of block queries and their arrival counters
  float* part_m; float* part_l; float* part_o; int* counters; int max_chunks;
  int32_t* status;
  int blk_to_state;          // block-row units write the merged state (m, l, O~) of their rows to `st` instead
                             // of normalised rows to `out` (first launch of an incremental advance)
  int st_tma;                // build: `st.o` is the buffer the cached-state tensor map was encoded for, so full row tiles
                             // may leave through bulk tensor stores (one-plane operands)
  int pair_chunks;           // host only: a step whose block-row units all have two key chunks, as pairs of CTAs
                             // (thread-block clusters of two) that merge through distributed shared memory
  int no_pdl;                // host only: launch the ordinary way (experiment knob)
  int split;                 // host only: rotated Q', K' are split bf16 planes (which kernel instantiation runs)
  // optional (lacache_set_span_ring): two device words of this launch; every CTA folds the global
  // nanosecond timer into them at entry (minimum) and at exit (maximum)
  unsigned long long* span;
};

struct SampleArgs {
  const void* logits; int dtype;   // [n_tokens, vocab], bf16 or fp32
  int n_tokens, vocab;
  const int32_t* rows; int n_rows; // the rows to sample (device)
  int splits, slice;               // CTAs per row and vocabulary entries per CTA (splits * slice >= vocab)
  int vector_ok;                   // rows start on 16-byte boundaries and `slice` is a multiple of the vector width
  float* part; int* counters;      // [n_rows][splits][4] partial results, [n_rows] arrival counters (zero between launches)
  float* conf; int32_t* token; float* lse;   // [n_rows]; lse may be null
  int32_t* status;
};
cudaError_t sample_rows(const SampleArgs& a, cudaStream_t s);

struct ExportArgs {
  RotBuffers rot; StateBuffers st;
  float* m; float* l; float* o;          // token-major outputs (may be null)
  float* q_rot; float* k_rot; float* v;  // token-major outputs (may be null)
};

// Partial states [B][Hq][max_chunks][block_len] (the layout the step kernel's block-row units write) of
// `tab[2 b + 1]` key chunks per sequence b, merged into the state of rows tab[2 b] ... of every head.
struct ChunkMergeArgs {
  const float* part_m; const float* part_l; const float* part_o; int max_chunks;
  const int32_t* tab;
  StateBuffers st;
  int no_pdl;   // host only: launch the ordinary way
};
cudaError_t merge_chunk_states(const Geometry& g, const ChunkMergeArgs& a, cudaStream_t s);

// ---- launchers implemented by the kernel files -----------------------------
// Each returns the cudaError_t of the launch (cudaGetLastError()).
// engine: LACACHE_ENGINE_SIMT or LACACHE_ENGINE_TCGEN05 (selects the storage
// format of the rotated planes).
cudaError_t rope_write(const Geometry& g, const RopeArgs& a, int engine, cudaStream_t s);
cudaError_t export_buffers(const Geometry& g, const ExportArgs& a, int engine, cudaStream_t s);

cudaError_t simt_attention(const Geometry& g, const AttnArgs& a, cudaStream_t s);
cudaError_t simt_prepare();  // function attributes

struct TcMaps;  // opaque set of TMA descriptors, defined in lacache_tc.cu
cudaError_t tc_attention(const Geometry& g, const AttnArgs& a, const TcMaps* maps, cudaStream_t s);
cudaError_t tc_prepare();
// builds TMA descriptors for a rotated buffer set; returns nullptr and fills
// err on failure
TcMaps* tc_make_maps(const Geometry& g, const RotBuffers& rot, float* state_o, bool split, char* err, int errlen);
// (re)encodes the descriptor of the caller's output buffer when it changed
bool tc_set_out(TcMaps* m, const Geometry& g, float* out, bool out_bf16, char* err, int errlen);
void tc_free_maps(TcMaps* m);

// token-wise producer (lacache_qkv.cu): the scratch rows the *_tokens entry points project into,
// and its head configuration (returns head_dim)
void qkv_scratch(lacache_qkv* p, bool block, void** q, void** k, void** v);
int qkv_heads(const lacache_qkv* p, int* hq, int* hkv, int* max_tokens);
// lacache_qkv_project with a scatter: input token t is written to output row dst_rows[t] (null: t)
// early_inputs: token_ids / hidden were complete before the grid ahead in the stream was enqueued, so the
// norm kernel may read them while that grid still runs (it waits for it at its end instead).
lacache_status qkv_project_rows(lacache_qkv* p, const int32_t* token_ids, const void* hidden, int n_tokens, void* q,
                                void* k, void* v, void* h_out, const int32_t* dst_rows, int max_rows, bool early_inputs,
                                void* stream);
// which context's tokens the all-token scratch holds (set by a full projection)
void qkv_set_full_owner(lacache_qkv* p, const void* ctx, int n_tokens);
bool qkv_full_owner_is(const lacache_qkv* p, const void* ctx, int n_tokens);

constexpr int SIMT_ROWS = 32;    // query rows per SIMT work item
constexpr int TC_ROWS = 128;     // query rows per tcgen05 work item
// keys per tile of the tcgen05 stream role: 96 with split operands (two stages of {K hi, K lo} and of V fit
// beside the Q tile), 128 with plain ones
constexpr int TC_KEYS_SPLIT = 96;
constexpr int TC_KEYS_PLAIN = 128;
inline int tc_keys(bool split) { return split ? TC_KEYS_SPLIT : TC_KEYS_PLAIN; }
constexpr int TC_MAX_BLOCK = 64;
constexpr int TC_DEEP_MAX_UNITS = 512;  // units per CTA the pipelined merge role can tabulate // largest block length the tcgen05 merge role handles

}  // namespace lacache
