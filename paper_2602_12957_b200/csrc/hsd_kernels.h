// Host-side launchers of the library's kernels (one translation unit per kernel family).
#pragma once

#include "hsd_common.cuh"

namespace hsd {

typedef __nv_bfloat16 bf16;

constexpr int kMaxDevices = 64;    // device ordinals the per-device launch state is kept for

struct ModelDims {
  int n_layers, d, Hq, Hkv, D, ffn, V, qkv_out, group;
  float rope_base, eps;
};

// The paged KV cache as the kernels see it.
struct KvView {
  bf16* k_pool;
  bf16* v_pool;
  int n_blocks;
  const int* block_table;
  int max_blocks;
  int* seq_lens;
  int n_slots;
};

// One launch path for every kernel: with `pdl` the launch carries the programmatic-stream-serialization
// attribute, so the kernel may start while its predecessor in the stream drains; such a kernel executes
// griddepcontrol.wait before it touches anything the predecessor wrote (or anything that is read by it).
template <typename... KArgs, typename... Args>
inline int launch_kernel(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, bool pdl,
                         Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...) == cudaSuccess ? 0 : -1;
}

enum KernelClass {
  KC_SETUP = 0, KC_EMBED, KC_RMSNORM, KC_GEMM_QKV, KC_ROPE_KV, KC_ATTN, KC_ATTN_COMBINE, KC_GEMM_O, KC_GEMM_GATEUP,
  KC_GEMM_DOWN, KC_LMHEAD, KC_ACCEPT, KC_COMMIT, KC_DEBUG, KC_COUNT
};
const char* kernel_class_name(int kc);

// ---- small kernels (hsd_small.cu) ---------------------------------------------------------------
struct SetupArgs {
  int n_seqs, total_q, max_q_len, vocab, tokens_per_tile;
  const int* cu_q;          // dev [S+1]
  const int* tokens;        // dev [T] or nullptr (page mode)
  const int* pending;       // dev [1] page mode: token of row 0
  const int* draft;         // dev [T-1] page mode: tokens of rows 1..
  const int* seq_slots;     // dev [S] or nullptr
  const int* parent;        // dev [T] or nullptr: candidate trees, parent row within the sequence (-1 for row 0)
  int slot_base;            // slot of sequence 0 when seq_slots == nullptr
  int allow_embed_rows;     // prefill: token id < 0 means "use the embeds row"
  float rope_base;
  int head_dim;
};
// `pdl` (here and below): launch with programmatic stream serialization; these kernels wait for their
// predecessor at their first instruction, so the flag only hides launch latency.
void launch_setup_rows(cudaStream_t st, const SetupArgs& a, const KvView& kv, const RowMeta& rm, int* status,
                       int* tile_count, bool pdl);
void launch_embed(cudaStream_t st, const RowMeta& rm, const bf16* table, const bf16* embeds, float* x, int T, int d,
                  const int* status, bool pdl);
// h[r] = bf16(rmsnorm(x[src]) * gain), src = sel_rows ? sel_rows[r] : r.  The gather form (sel_rows != nullptr) writes
// nothing when *status is set or src is outside [0, src_rows): the index comes from an earlier kernel of the step.
void launch_rmsnorm(cudaStream_t st, const float* x, const bf16* gain, bf16* h, int rows, int d, float eps,
                    const int* sel_rows, int src_rows, const int* status, bool pdl);
// last row of every sequence (prefill's LM-head rows); -1 for every sequence when *status is set
void launch_select_last_rows(cudaStream_t st, const RowMeta& rm, int n_seqs, int* sel_rows, const int* status, bool pdl);
// q_norm / k_norm: per-head RMSNorm gains applied before the rotation, or nullptr
void launch_rope_kvwrite(cudaStream_t st, const float* qkv, const RowMeta& rm, const KvView& kv, const ModelDims& md,
                         int layer, bf16* q, int T, const int* status, const bf16* q_norm, const bf16* k_norm);
void launch_attn_simt(cudaStream_t st, const bf16* q, const RowMeta& rm, const KvView& kv, const ModelDims& md,
                      int layer, bf16* out, int T, const int* status);
struct AcceptArgs {
  int n_seqs, max_q_len;
  float log_tau;
  const unsigned long long* row_best;
  const float* zdraft;
  int* accept_len;
  int* emit_tokens;
  int* n_emit;
  int* row_argmax;     // optional outputs
  float* row_zmax;
  float* row_zdraft;
};
void launch_accept(cudaStream_t st, const AcceptArgs& a, const RowMeta& rm, const int* status, bool pdl);
// Greedy traversal of candidate trees (Eq. 9-12).  LM-head row r < T holds the argmax at node r, row T + r the
// logit of node r's own token under its parent's distribution.
struct TreeAcceptArgs {
  int n_seqs, max_q_len, total_q;
  float log_tau;
  const int* parent;
  const unsigned long long* row_best;   // [2T]
  const float* zdraft;                  // [2T]
  int* accept_len;
  int* emit_tokens;
  int* n_emit;
  int* accept_rows;    // [S, max_q_len] rows of the accepted path after the root
  int* row_argmax;     // optional outputs, [T]
  float* row_zmax;
  float* row_zchild;
};
void launch_tree_accept(cudaStream_t st, const TreeAcceptArgs& a, const RowMeta& rm, const int* status, bool pdl);
// Moves the K/V rows of an accepted tree path (cache rows L + accept_rows[d-1]) to rows L + d, every layer and head.
void launch_tree_compact(cudaStream_t st, const KvView& kv, int n_layers, int n_kv_heads, int head_dim, int n_seqs, const int* seq_slots,
                         const int* accept_len, const int* accept_rows, int max_q_len, bool pdl);
// Draft-target matching + prefix-tree packing on the device (Eq. 5-7)
struct DsvArgs {
  int n_seqs, window_n, max_rows, emit_stride, total_draft_tokens, n_drafts;
  int* window;               // [S, n] inout
  const int* emit_tokens;    // [S, emit_stride] or nullptr
  const int* n_emit;         // [S] or nullptr
  const int* draft_tokens;
  const int* draft_off;      // [n_drafts + 1]
  const int* seq_draft_off;  // [owners + 1]
  const int* seq_map;        // [S] or nullptr: sequence i matches against the drafts of owner seq_map[i] (-1: none)
  int n_owners;              // entries of seq_draft_off minus one (used with seq_map)
  int* q_tokens;             // [S * max_rows]
  int* parent;               // [S * max_rows]
  int* cu_q;                 // [S + 1]
  int* n_rows;               // [S]
};
void launch_dsv_build(cudaStream_t st, const DsvArgs& a, bool pdl);
// Decode-loop bookkeeping between two steps of a lane batch (Sec. 3.1): append what every lane's sequence emitted,
// retire finished sequences, hand their lanes to waiting ones.  Mirrors hsd_stage in the public header.
struct StageDev {
  int n_lanes, n_seqs, window_n, out_stride, idle_slot;
  int* lane_seq;
  int* lane_slot;
  int* window;
  const int* first_token;
  const int* seq_slot;
  const int* max_new;
  int* out_tokens;
  int* out_len;
  int* seq_steps;
  int* seq_accepted;
  int* counters;
};
void launch_stage_begin(cudaStream_t st, const StageDev& sd, const KvView& kv, bool pdl);
void launch_stage_advance(cudaStream_t st, const StageDev& sd, const KvView& kv, const int* accept_len,
                          const int* emit_tokens, const int* n_emit, int emit_stride, bool pdl);
void launch_stage_aggregate(cudaStream_t st, const StageDev& sd, int* draft_tokens, int capacity, int* draft_off, bool pdl);
void launch_first_token(cudaStream_t st, const unsigned long long* row_best, int n_seqs, int* first_token,
                        const RowMeta& rm, const KvView& kv, const int* status, bool pdl);
void launch_commit(cudaStream_t st, const KvView& kv, int n_seqs, const int* seq_slots, const int* accept_len,
                   int* blocks_in_use, bool pdl);
void launch_clear_best(cudaStream_t st, unsigned long long* row_best, float* zdraft, int rows, bool pdl);
void launch_unpack_best(cudaStream_t st, const unsigned long long* row_best, int rows, int* argmax, float* zmax,
                        bool pdl);

// ---- attention plan (hsd_attn_sm100.cu): made once per step on the device, read by every layer's launch ----
constexpr int kAttnMaxSplits = 8;      // most KV slices one q-tile is cut into
struct AttnPlan {
  int4* items;      // two int4 per (q-tile, slice) item, longest first: {first packed row, position of the first
                    // token, tokens, KV slot}, {first | (last + 1) << 16 KV tile, slice | slices << 8 | first token of the q-tile within its sequence << 16,
                    // q-tile, KV tiles}
  int4* items_unsorted;   // the same list in creation order (scratch of the plan kernel)
  int* n_items;
  int* tile_seq;    // [max_tiles] sequence of a q-tile
  int* tile_nkv;    // [max_tiles] KV tiles it can see
  int* counters;    // [max_tiles, n_kv_heads] slices that have delivered their partial
  int4* first;      // [grid CTAs][3]: the item a CTA of the attention grid starts with, ready to use: the item's two
                    // words, then {item x kv head index (-1: none), kv head, first two physical KV blocks}
  int n_kv_heads;
  int grid;         // CTAs of the attention launches this plan is made for
};
void launch_attn_plan(cudaStream_t st, const RowMeta& rm, const AttnPlan& pl, const KvView& kv, int n_seqs,
                      int tokens_per_tile, int target_items, int min_chunk, const int* tile_count, const int* status,
                      bool pdl);
int launch_attn_sm100(cudaStream_t st, const CUtensorMap& tmQ, const CUtensorMap& tmK, const CUtensorMap& tmV,
                      const AttnPlan& plan, const KvView& kv, const ModelDims& md, int layer, bf16* out, int n_sms,
                      int device, int* status, float* split_ws, const uint4* anc, bool pdl);

// ---- plain SIMT GEMM (hsd_gemm_simt.cu): the debug cross-check and hsd_debug_logits --------------
enum GemmMode { GM_STORE_BF16 = 0, GM_ADD_F32 = 1, GM_SWIGLU = 2, GM_STORE_F32 = 3, GM_ARGMAX = 4 };
struct GemmOut {
  void* C;                         // bf16 / fp32 output (modes 0-3), leading dimension ldc
  int ldc;
  unsigned long long* row_best;    // mode 4
  float* zdraft;                   // mode 4
  const int* row_next;             // mode 4 (nullptr = no draft-token capture)
};
void launch_gemm_simt(cudaStream_t st, const bf16* A, const bf16* W, int M, int n_out, int K, int mode,
                      const GemmOut& out);

// ---- tcgen05 GEMM (hsd_gemm_sm100.cu) ------------------------------------------------------------
// Encode a 2-D bf16 row-major [rows, cols] tensor map with a {64, box_rows} box and 128-byte swizzle.
int make_tmap_2d(CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows);
// Same for fp32 with a {32, box_rows} box (128-byte rows): the residual stream as a TMA reduce-add target.
int make_tmap_2d_f32(CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows);
// The three maps of one weight matrix, box heights 32 / 64 / 128 rows = half a tile of width 64 / 128 / 256.
struct WeightMaps {
  CUtensorMap m[3];
};
int make_weight_tmaps(WeightMaps* w, const void* base, uint64_t rows, uint64_t cols);
int make_tmap_3d(CUtensorMap* map, const void* base, uint64_t d0, uint64_t d1, uint64_t d2, uint64_t stride1_bytes,
                 uint64_t stride2_bytes, uint32_t b0, uint32_t b1, uint32_t b2);
int tma_init();   // resolves cuTensorMapEncodeTiled; 0 on success

struct QkvEpilogue {      // fused RoPE + paged KV write (QKV projection)
  const int* row_kv;
  int kv_rows;            // rows of one layer of the pool (blocks x 64): a physical row outside it is never written
  const float2* rope_cs;
  bf16* q_out;            // [T, Hq*D]
  bf16* k_pool_layer;     // layer base of the K pool
  bf16* v_pool_layer;
  int Hq, Hkv, D;         // D = head_dim (64 or 128)
  const bf16* q_norm;     // per-head RMSNorm gains [D] of q and k before the rotation, or nullptr (none)
  const bf16* k_norm;
  float eps;
};
struct GemmSm100Args {
  CUtensorMap tmA;             // activations, box {64, 128}
  const WeightMaps* tmB;       // weights
  CUtensorMap tmC;             // output through TMA: bf16 box {64, 32} (store) or fp32 box {32, 32} (reduce-add);
                               // the q buffer for GS_QKV_ROPE; unused for GS_ARGMAX
  int M, n_out, K, mode;
  GemmOut out;
  QkvEpilogue qkv;
  int* status;
  int n_sms;
  int device;                  // CUDA device ordinal of the launch (per-device kernel attributes)
  int max_splits;              // GS_ADD_F32: most K slices per tile (1 = none; slices add in arrival order)
  bool pdl;                    // launch with programmatic stream serialization
  int pair;                    // CTA pairs (clusters of two sharing a 256-row tile) may be used
  int force_bn, force_splits;  // tests: tile width (512 = CTA pair) / K slices instead of the model's choice (0 = choose)
};
enum GemmSm100Mode { GS_STORE_BF16 = 0, GS_ADD_F32 = 1, GS_SWIGLU = 2, GS_ARGMAX = 4, GS_QKV_ROPE = 5, GS_QKV_ROPE128 = 6 };
int launch_gemm_sm100(cudaStream_t st, const GemmSm100Args& a);

}  // namespace hsd
