/*
 * hsd.h — C ABI of the B200 (sm_100a) draft-verification step of Hierarchical Speculative Decoding.
 *
 * One call = one step of the verification operator y_hat = SpecDecode(p_theta, z, Y~) (paper Eq. 1):
 * the target decoder scores, in a single forward over a cached prefix, every token of one or many drafts
 * (Eq. 8, chain-shaped candidate tree: a draft token attends to the accepted tokens and, causally, to the
 * draft tokens before it), takes the full-vocabulary argmax per row (Eq. 10), accepts the longest prefix of
 * the draft that matches it (Eq. 9 and 11 with one candidate per node and tau = 1; with log_tau < 0 the
 * thresholded test of Eq. 11), and emits the accepted tokens plus the correction / bonus token (Eq. 12).
 * KV maintenance after the step (commit of the accepted rows, rollback of the rest; counted in T_decode,
 * Sec. 4.2) is a separate call.
 *
 * Beside the chain form there is the paper's general operator and the loop around it: hsd_dsv_build (reference
 * window, matching, prefix tree and its packing, Eq. 5-7), hsd_verify_tree / hsd_kv_commit_tree (candidate
 * trees under the ancestry mask, greedy traversal, compaction of the accepted path, Eq. 8-12), and
 * hsd_stage_begin / hsd_stage_advance / hsd_stage_aggregate (outputs, retirement and lane hand-over of the two
 * stages and the page draft, Sec. 3.1, Eq. 2-4): a whole stage runs as stream-ordered calls of fixed shape,
 * with no host decision between steps.
 *
 * Conventions
 *  - All functions return an int status: HSD_OK (0) or a negative HSD_ERR_* code.  Nothing throws.
 *  - "dev" pointers are CUDA device pointers on the current device; "host" pointers are ordinary memory.
 *  - The library allocates NO device memory: weights, KV pool, block table, sequence lengths, workspace,
 *    inputs and outputs are owned by the caller and must stay alive until the stream work has finished.
 *    An hsd_ctx owns host memory only (configuration, tensor maps, profiling events).
 *  - Every compute call is asynchronous on the given cudaStream_t (passed as void*), performs no
 *    synchronisation and leaves its outputs on the device.
 *  - Pending-token convention: the most recently emitted token of a sequence has no K/V yet; it is query
 *    row 0 of the next step.  A k-token draft is therefore k+1 query rows, and full acceptance emits k+1
 *    tokens.
 *  - bf16 storage, fp32 accumulation, fp32 residual stream.
 *
 * Memory layouts (row-major, last index fastest)
 *  - Linear weights: bf16 [out_features, in_features]  (y = x W^T).
 *      w_qkv     [(n_heads + 2 n_kv_heads) * head_dim, d_model]   rows: q heads, k heads, v heads
 *      w_o       [d_model, n_heads * head_dim]
 *      w_gate_up [2 * d_ffn, d_model]                             rows: gate, then up
 *      w_down    [d_model, d_ffn]
 *      embed, lm_head [vocab, d_model];  *_norm [d_model] (bf16 gains)
 *  - Paged KV pool, block = kv_block (64) tokens:
 *      k_pool, v_pool bf16 [n_layers][n_blocks][n_kv_heads][64 tokens][head_dim]
 *    (one row of head_dim bf16 per token and kv head: 128 or 256 bytes; a (block, kv head) tile is contiguous)
 *    block_table int32 [n_slots, max_blocks_per_seq]: physical block of logical block j of slot s.
 *    seq_lens int32 [n_slots]: committed K/V rows per slot.
 *  - Packed query tokens: q_tokens[cu_q[i] .. cu_q[i+1]) = [pending_i, d_i1 .. d_ik].
 */
#ifndef HSD_H_
#define HSD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define HSD_API __attribute__((visibility("default")))
#else
#define HSD_API
#endif

#define HSD_OK 0
#define HSD_ERR_INVALID_ARG (-1)   /* null pointer, negative size, inconsistent arguments            */
#define HSD_ERR_SHAPE (-2)         /* model shape not supported by the kernels                        */
#define HSD_ERR_TOO_LONG (-3)      /* a sequence has more query rows than HSD_MAX_Q_LEN               */
#define HSD_ERR_WORKSPACE (-4)     /* workspace too small or misaligned                               */
#define HSD_ERR_KV_CAPACITY (-5)   /* declared KV capacity cannot hold the step                       */
#define HSD_ERR_CUDA (-6)          /* a CUDA call failed; see hsd_last_cuda_error                     */
#define HSD_ERR_DEVICE_CHECK (-7)  /* a device-side check tripped; see hsd_device_status              */
#define HSD_ERR_NO_DEVICE (-8)     /* no usable sm_100 device                                         */

#define HSD_MAX_Q_LEN 4097         /* most query rows one sequence may have in a verify call          */
#define HSD_MAX_TREE_ROWS 128      /* most rows (root included) of one sequence in hsd_verify_tree    */
#define HSD_MAX_WINDOW 8           /* longest reference window hsd_dsv_build takes (the paper uses 3)   */
#define HSD_DSV_MAX_CANDIDATES 64  /* candidate suffixes per sequence; later matches are ignored        */
#define HSD_KV_BLOCK 64

/* hsd_model_config.flags */
#define HSD_FLAG_SIMT_DEBUG 1      /* run the plain SIMT kernels instead of the tensor-core kernels;
                                      a slow cross-check for debugging, never a fallback              */
#define HSD_FLAG_SIMT_ATTENTION 2  /* debugging: only the attention runs through its plain kernel     */
#define HSD_FLAG_DETERMINISTIC 4   /* no split-K in the residual-add projections (their K slices add into
                                      the fp32 residual in arrival order, so results can differ in the last
                                      bit from run to run) and no KV slicing in the attention (where the cuts
                                      fall depends on what else is in the batch): with this flag every run is
                                      bit-identical and a row's result does not depend on the batch around it;
                                      a single sequence over a long context then runs on few SMs            */
#define HSD_FLAG_NO_PAIR 16        /* debugging: no CTA-pair (cluster of two) GEMM tiles                        */
#define HSD_FLAG_NO_HOST_GRAPH 32  /* hsd_verify_regions_host launches its kernels one by one, never as a CUDA graph */
#define HSD_FLAG_NO_PDL 8          /* debugging: plain stream-ordered launches (no programmatic dependent
                                      launch overlap between consecutive kernels)                       */

typedef struct hsd_ctx hsd_ctx;

typedef struct {
  int n_layers, d_model, n_heads, n_kv_heads, head_dim, d_ffn, vocab;
  float rope_base;   /* rotary base (10000)                                                           */
  float rms_eps;     /* RMSNorm epsilon                                                               */
  int kv_block;      /* must be 64                                                                    */
  int flags;         /* HSD_FLAG_*                                                                    */
  int qk_norm;       /* 1: per-head RMSNorm (over head_dim, rms_eps) of q and k before the rotary embedding,
                        with the gains hsd_weights.q_norm / k_norm (Qwen3-style decoders); 0: none     */
} hsd_model_config;

/* Device pointers to bf16 weights.  The per-layer members are HOST arrays of n_layers device pointers. */
typedef struct {
  const void *embed, *lm_head, *final_norm;
  const void *const *attn_norm, *const *w_qkv, *const *w_o;
  const void *const *ffn_norm, *const *w_gate_up, *const *w_down;
  const void *const *q_norm, *const *k_norm;   /* bf16 [head_dim] per layer; read only when qk_norm = 1, else may be NULL */
} hsd_weights;

/* Caller-owned paged KV cache.  All pointers are device pointers.
 * k_pool and v_pool must hold FINITE values everywhere before the first call (zero them once at allocation): a key the
 * mask hides still enters the second attention product as 0 * v, which is 0 only for finite v, so an Inf or NaN bit
 * pattern left in a row that was never written would turn that tile's outputs into NaN. */
typedef struct {
  void *k_pool, *v_pool;
  int n_blocks;               /* physical blocks per layer                                            */
  const int *block_table;     /* [n_slots, max_blocks_per_seq]                                        */
  int max_blocks_per_seq;
  int *seq_lens;              /* [n_slots], updated by hsd_prefill and hsd_kv_commit                  */
  int n_slots;
} hsd_kv;

HSD_API const char *hsd_status_string(int status);

/* Create a context for one model on the current device.  Copies the configuration and the weight POINTERS
 * (not the weights) and builds the TMA tensor maps of the weights.  Errors: INVALID_ARG, SHAPE (requires
 * head_dim 64 or 128 (128 not together with the HSD_FLAG_SIMT_* cross-check kernels), kv_block == 64, n_heads a multiple of n_kv_heads with a ratio that divides 128, d_model one of
 * 128, 256, 512, 1024, 2048, 4096, d_ffn and vocab multiples of 64),
 * NO_DEVICE, CUDA.  No stream work is issued. */
HSD_API int hsd_create(const hsd_model_config *cfg, const hsd_weights *w, hsd_ctx **out);
HSD_API int hsd_destroy(hsd_ctx *ctx);

/* Bytes of device workspace a call with at most max_total_q packed query rows and max_seqs sequences
 * needs.  The workspace must be 1024-byte aligned.  Its first 64 bytes hold the device status words
 * (hsd_device_status); the rest is scratch that keeps nothing between calls. */
HSD_API size_t hsd_workspace_bytes(const hsd_ctx *ctx, int max_total_q, int max_seqs);

/* Support call, outside the decode loop (Sec. 4.2 excludes prefill from T_decode): run prefix rows through
 * the decoder, write their K/V into the pool at positions seq_lens[slot] .., advance seq_lens by the row
 * count, and return each sequence's greedy next token (the first pending token).
 *   cu_len    dev int32 [n_seqs+1]  row offsets of the sequences in the packed input
 *   embeds    dev bf16 [total_rows, d_model] or NULL; row r is used where token_ids[r] < 0 (visual rows)
 *   token_ids dev int32 [total_rows]; >= 0 selects a row of the embedding table
 *   seq_slots dev int32 [n_seqs] or NULL (= slots 0 .. n_seqs-1)
 *   first_token dev int32 [n_seqs] out
 *   total_rows, max_len: host copies of cu_len[n_seqs] and max_i(cu_len[i+1]-cu_len[i]) (max_len <= 32768)
 */
HSD_API int hsd_prefill(hsd_ctx *ctx, const hsd_kv *kv, int n_seqs, const int *cu_len, const void *embeds,
                const int *token_ids, const int *seq_slots, int total_rows, int max_len, int *first_token,
                void *workspace, size_t ws_bytes, void *cuda_stream);

/* Stage 1, region-level verification (Eq. 2): a varlen batch of independent sequences, each
 * [pending, draft].  Writes the speculative K/V rows of all query rows in place at positions
 * seq_lens[slot] .. seq_lens[slot]+k (nothing is committed; seq_lens is not changed).
 *   cu_q, q_tokens  dev int32 [n_seqs+1], [total_q]
 *   seq_slots       dev int32 [n_seqs] or NULL (= slots 0 .. n_seqs-1)
 *   max_q_len, total_q  host copies of max_i(k_i+1) (<= HSD_MAX_Q_LEN) and cu_q[n_seqs]
 *   log_tau         0 = exact greedy match (the contract); < 0 = accept d iff z[d] - z_max >= log_tau
 *   accept_len      dev int32 [n_seqs] out: accepted draft tokens a_i
 *   emit_tokens     dev int32 [n_seqs, max_q_len] out: d_i1..d_ia, then the correction/bonus token
 *   n_emit          dev int32 [n_seqs] out: a_i + 1
 *   row_argmax      dev int32 [total_q] out or NULL: u_hat per row (lowest id on ties)
 *   row_zmax        dev fp32  [total_q] out or NULL: its logit
 *   row_zdraft      dev fp32  [total_q] out or NULL: logit of the row's next draft token (NaN on a
 *                   sequence's last row)
 * Device-side checks (cu_q monotone, q_i <= max_q_len, token ids in range, block table entries in range,
 * seq_len + q_i within max_blocks_per_seq * 64) set the status words and turn the step into a no-op. */
HSD_API int hsd_verify_regions(hsd_ctx *ctx, const hsd_kv *kv, int n_seqs, const int *cu_q, const int *q_tokens,
                       const int *seq_slots, int max_q_len, int total_q, float log_tau, int *accept_len,
                       int *emit_tokens, int *n_emit, int *row_argmax, float *row_zmax, float *row_zdraft,
                       void *workspace, size_t ws_bytes, void *cuda_stream);

/* Stage 2, page-level verification (Eq. 4): one sequence, one chunk of the page draft.
 *   pending_token   dev int32 [1]: the sequence's pending token (e.g. the last entry of the previous
 *                   call's emit_tokens)
 *   draft_chunk     dev int32 [chunk_len], chunk_len + 1 <= HSD_MAX_Q_LEN
 *   outputs as above with n_seqs = 1, max_q_len = chunk_len + 1. */
HSD_API int hsd_verify_page(hsd_ctx *ctx, const hsd_kv *kv, int seq_slot, const int *pending_token,
                    const int *draft_chunk, int chunk_len, float log_tau, int *accept_len, int *emit_tokens,
                    int *n_emit, int *row_argmax, float *row_zmax, float *row_zdraft, void *workspace,
                    size_t ws_bytes, void *cuda_stream);

/* One verification step over candidate TREES (Sec. 3.2: prefix tree T of Eq. 7 packed into one sequence, the
 * tree-ancestry mask of Fig. 2(c), greedy traversal of Eq. 9-12).  Per sequence the packed rows are
 * [pending token (the root), node 1, .., node k] in an order that puts every parent before its children;
 *   parent          dev int32 [total_q]: the parent's row index WITHIN the sequence, -1 for row 0; -2 marks a
 *                   padding row (no parent, no children: it sees the committed context and itself, nothing can
 *                   move to it; hsd_dsv_build pads with such rows to keep shapes fixed)
 *   max_q_len       at most HSD_MAX_TREE_ROWS rows per sequence (root included; the paper packs <= 128 tokens)
 * A node's rotary position is committed length + depth; it attends to the committed context, itself and its
 * ancestors.  Traversal from the root: at node s, u_hat = argmax over the vocabulary (lowest id on ties), u* = the
 * child of s with the highest logit (log_tau = 0: the child that carries u_hat); move to it iff
 * z[u*] - z[u_hat] >= log_tau; stop when the test fails or s is a leaf; emitted = tokens of the path, then u_hat.
 *   accept_len      dev int32 [n_seqs] out: length of the accepted path
 *   emit_tokens     dev int32 [n_seqs, max_q_len] out, n_emit = accept_len + 1
 *   accept_rows     dev int32 [n_seqs, max_q_len] out: rows of the accepted path after the root
 *   row_argmax, row_zmax   dev [total_q] out or NULL, as in hsd_verify_regions
 *   row_zchild      dev fp32 [total_q] out or NULL: the logit of the row's own token under its parent's
 *                   distribution (NaN on row 0)
 * The K/V rows of ALL nodes are written at cache rows committed length + row index; hsd_kv_commit_tree keeps the
 * accepted ones.  The workspace must be sized for 2 * total_q rows (the LM head evaluates every node once for its
 * argmax and once more, through its parent, for its own token).  A parent pointer that does not name an earlier row
 * sets device status 7 and turns the step into a no-op.  Errors otherwise as hsd_verify_regions; contexts created
 * with a SIMT debug flag return HSD_ERR_INVALID_ARG. */
HSD_API int hsd_verify_tree(hsd_ctx *ctx, const hsd_kv *kv, int n_seqs, const int *cu_q, const int *q_tokens,
                    const int *parent, const int *seq_slots, int max_q_len, int total_q, float log_tau,
                    int *accept_len, int *emit_tokens, int *n_emit, int *accept_rows, int *row_argmax, float *row_zmax,
                    float *row_zchild, void *workspace, size_t ws_bytes, void *cuda_stream);

/* Draft-target matching and prefix-tree packing on the device (Sec. 3.2, Eq. 5-7), so that a decode loop of
 * hsd_dsv_build -> hsd_verify_tree -> hsd_kv_commit_tree has fixed shapes and needs no host decision between steps.
 *   window          dev int32 [n_seqs, window_n] INOUT: the window_n (<= HSD_MAX_WINDOW) most recent accepted
 *                   tokens of every sequence, oldest first; a negative entry means "not that many tokens yet" (no
 *                   match is attempted then); the last entry is the pending token and must be a valid id
 *   emit_tokens, n_emit   dev int32 [n_seqs, emit_stride], [n_seqs] or both NULL: the tokens the previous step
 *                   emitted; they are appended to the window before matching (and the window is written back)
 *   draft_tokens    dev int32 [total_draft_tokens], all drafts concatenated;  draft_off dev int32 [n_drafts + 1]
 *                   their offsets;  seq_draft_off dev int32 [n_seqs + 1]: sequence i owns drafts
 *                   seq_draft_off[i] .. seq_draft_off[i+1] - 1.  n_drafts and total_draft_tokens are host copies of
 *                   the array sizes: the kernel clamps every offset it reads to them, so malformed offsets shorten
 *                   or drop drafts but never read outside the arrays
 *   max_rows        rows every sequence gets in the packed output (<= HSD_MAX_TREE_ROWS; the paper packs 128)
 *   q_tokens, parent  dev int32 [n_seqs * max_rows] out: row 0 = the pending token (parent -1), then the tree's
 *                   nodes with their parent rows, then padding rows (the pending token again, parent -2) which
 *                   hsd_verify_tree treats as rows without parent or children
 *   cu_q            dev int32 [n_seqs + 1] out: i * max_rows;   n_rows dev int32 [n_seqs] out: 1 + nodes
 * Candidates: for every draft of the sequence and every position where the window occurs (Eq. 5), the non-empty
 * suffix after it (Eq. 6), in draft order then position order, at most HSD_DSV_MAX_CANDIDATES.  Tree (Eq. 7): one
 * node per distinct prefix, created level by level in candidate order while fewer than max_rows - 1 nodes exist; a
 * candidate whose next node cannot be created stops growing.  Pure integer work: results are exact.
 *   seq_map         dev int32 [n_seqs] or NULL: with a map, sequence i matches against the drafts of OWNER seq_map[i], i.e.
 *                   drafts seq_draft_off[seq_map[i]] .. seq_draft_off[seq_map[i] + 1] - 1 (lane batches: a lane serves
 *                   different sequences over time); an entry < 0 or >= n_owners means "no drafts".  n_owners = entries of
 *                   seq_draft_off minus one (host copy; ignored without a map, where it is n_seqs). */
HSD_API int hsd_dsv_build(hsd_ctx *ctx, int n_seqs, int window_n, int *window, const int *emit_tokens, const int *n_emit,
                  int emit_stride, const int *draft_tokens, int total_draft_tokens, const int *draft_off,
                  int n_drafts, const int *seq_draft_off, int max_rows, int *q_tokens, int *parent, int *cu_q,
                  int *n_rows, const int *seq_map, int n_owners, void *cuda_stream);

/* Decode loop over a LANE BATCH (Sec. 3.1): Stage 1 runs SpecDecode (Eq. 2) on all regions of a page "in parallel" until
 * every region's output is complete; Stage 2 (Eq. 4) is the same loop with one lane.  n_lanes lanes step together
 * (hsd_dsv_build -> hsd_verify_tree -> hsd_kv_commit_tree over the lanes, with seq_slots = lane_slot and seq_map =
 * lane_seq); a lane serves one sequence until its output has max_new tokens, then takes the next waiting sequence, so the
 * batch shape stays fixed while regions of different lengths come and go.  All decisions are taken on the device: the
 * host only polls counters[1] (sequences not finished) now and then.
 * All pointers are device pointers owned by the caller.
 *   lane_seq      [n_lanes]            sequence a lane serves, -1 = none (the lane then idles on KV slot idle_slot, whose
 *                                      length is reset to 0 after every step; give it room for one step's rows)
 *   lane_slot     [n_lanes]            KV slot of every lane for the next step (pass as seq_slots)
 *   window        [n_lanes, window_n]  reference window of every lane (pass to hsd_dsv_build WITHOUT emit_tokens: the
 *                                      advance call below has already taken the emitted tokens in)
 *   first_token   [n_seqs]             first token of every sequence (hsd_prefill's output): token 0 of its output and
 *                                      its first pending token
 *   seq_slot      [n_seqs] or NULL     KV slot of every sequence (NULL: slot = sequence index)
 *   max_new       [n_seqs]             output length of every sequence (the paper's parsers stop at their end token; the
 *                                      synthetic decoders have none, so lengths are given)
 *   out_tokens    [n_seqs, out_stride] outputs; out_len [n_seqs] tokens so far; seq_steps [n_seqs] verification steps
 *                                      spent; seq_accepted [n_seqs] accepted draft tokens (AAL = accepted / steps, Sec. 4.2)
 *   counters      [4]                  [0] next waiting sequence, [1] sequences not finished, [2] steps taken */
typedef struct {
  int n_lanes, n_seqs, window_n, out_stride, idle_slot;
  int *lane_seq, *lane_slot, *window;
  const int *first_token, *seq_slot, *max_new;
  int *out_tokens, *out_len, *seq_steps, *seq_accepted, *counters;
} hsd_stage;

/* Start a lane batch: every output gets its first token, lanes take the first sequences of the queue (in order), the
 * others wait.  Errors: INVALID_ARG (null pointers, n_lanes / n_seqs / out_stride < 1, window_n outside 1..HSD_MAX_WINDOW). */
HSD_API int hsd_stage_begin(hsd_ctx *ctx, const hsd_stage *stage, const hsd_kv *kv, void *cuda_stream);

/* Between two steps: append every lane's emitted tokens (emit_tokens [n_lanes, emit_stride], n_emit, accept_len: the
 * outputs of the step's hsd_verify_tree) to its sequence's output up to max_new, count the step and its accepted tokens,
 * rebuild the lane's window from the output's last tokens, retire finished sequences and give their lanes to the next
 * waiting ones (lanes in index order, queue order: deterministic).  A lane whose accept_len is -1 (the step failed a
 * device-side check) is left as it was. */
HSD_API int hsd_stage_advance(hsd_ctx *ctx, const hsd_stage *stage, const hsd_kv *kv, const int *accept_len,
                      const int *emit_tokens, const int *n_emit, int emit_stride, void *cuda_stream);

/* The page draft (Eq. 3): all outputs concatenated into draft_tokens (dev int32 [capacity]) with draft_off (dev int32
 * [n_seqs + 1]) their offsets, in the layout hsd_dsv_build takes; outputs beyond `capacity` are cut. */
HSD_API int hsd_stage_aggregate(hsd_ctx *ctx, const hsd_stage *stage, int *draft_tokens, int capacity, int *draft_off,
                        void *cuda_stream);

/* KV maintenance after hsd_verify_tree (Sec. 4.2 counts it in the decode loop): in every layer the K/V rows of the
 * accepted path move from cache rows L + accept_rows[i][d-1] to rows L + d (d = 1..accept_len[i]; L = committed
 * length; the values already carry the rotary position L + d), then seq_lens[slot_i] += accept_len[i] + 1.
 * blocks_in_use as in hsd_kv_commit. */
HSD_API int hsd_kv_commit_tree(hsd_ctx *ctx, const hsd_kv *kv, int n_seqs, const int *seq_slots, const int *accept_len,
                       const int *accept_rows, int max_q_len, int *blocks_in_use, void *cuda_stream);

/* KV maintenance after a step: seq_lens[slot_i] += accept_len[i] + 1 (the pending row and the accepted
 * draft rows stay; rows after them are rolled back and will be overwritten by the next step).  The caller
 * may pass lengths other than the ones verify produced.  blocks_in_use (dev int32 [n_seqs] or NULL)
 * receives ceil(new_len / 64). */
HSD_API int hsd_kv_commit(hsd_ctx *ctx, const hsd_kv *kv, int n_seqs, const int *seq_slots, const int *accept_len,
                  int *blocks_in_use, void *cuda_stream);

/* Stage 1 with HOST buffers: the same step as hsd_verify_regions followed (if commit != 0) by hsd_kv_commit, for
 * callers whose drafts and results live in host memory (Eq. 2 and Eq. 12 end to end, including the transfers the
 * paper counts in T_decode, Sec. 4.2).
 *   cu_q, q_tokens        HOST int32 [n_seqs+1], [cu_q[n_seqs]] (pinned memory makes the copies asynchronous)
 *   seq_slots             dev int32 [n_seqs] or NULL, as above
 *   accept_len, n_emit    HOST int32 [n_seqs] out
 *   emit_tokens           HOST int32 [n_seqs, max_q_len] out, max_q_len = max_i(cu_q[i+1]-cu_q[i]), also
 *                         returned through max_q_len_out (may be NULL); the buffer must hold n_seqs * max_q_len ints
 * Copies the inputs into staging areas inside `workspace`, runs the step on the stream, copies the results back and
 * SYNCHRONISES the stream before returning; a device-side check that tripped is returned as HSD_ERR_DEVICE_CHECK.
 * The transfers go through pinned staging owned by the context.  When the same call shape (every argument but the
 * contents of cu_q / q_tokens, with equal n_seqs, total and longest query length) comes a second time on a stream
 * other than the default one, the whole step is captured once into a CUDA graph and replayed from then on, which
 * removes the per-kernel launch cost from the decode loop (HSD_FLAG_NO_HOST_GRAPH turns this off).  The caller
 * must not be capturing the stream itself.
 * Errors otherwise as hsd_verify_regions. */
HSD_API int hsd_verify_regions_host(hsd_ctx *ctx, const hsd_kv *kv, int n_seqs, const int *cu_q, const int *q_tokens,
                            const int *seq_slots, float log_tau, int commit, int *accept_len, int *emit_tokens,
                            int *n_emit, int *max_q_len_out, void *workspace, size_t ws_bytes, void *cuda_stream);

/* Device status words written by the last call that used `workspace` (synchronises the stream).
 * status[0] = 0 if every device-side check passed, else a code (1 cu_q not monotone, 2 sequence too long,
 * 3 token id out of range, 4 KV capacity, 5 block table entry out of range, 6 a bounded wait gave up,
 * 7 a tree's parent pointer does not name an earlier row of its sequence);
 * status[1] = index of the offending sequence or row. */
HSD_API int hsd_device_status(hsd_ctx *ctx, const void *workspace, void *cuda_stream, int status[4]);

/* cudaError_t of the last failed CUDA call in this context (0 if none). */
HSD_API int hsd_last_cuda_error(const hsd_ctx *ctx);

/* Kernels launched by this context so far. */
HSD_API long long hsd_launch_count(const hsd_ctx *ctx);

/* Per-kernel-class timing with CUDA events on the launching stream.  enable != 0 starts recording (resets
 * the totals); hsd_profile_read synchronises the recorded events and fills up to `cap` entries of
 * names[i] (static strings), total_ms[i], launches[i]; returns the number of classes or a negative status.
 * Recording adds two event records per launch; leave it off when timing whole steps. */
HSD_API int hsd_profile_enable(hsd_ctx *ctx, int enable);
HSD_API int hsd_profile_read(hsd_ctx *ctx, int cap, const char **names, double *total_ms, long long *launches);

/* Test-only: full logits of the query rows of the LAST verify call that used `workspace`
 * (fp32 [total_q, vocab], row-major); total_q and n_seqs must be that call's.  Slow plain kernel. */
HSD_API int hsd_debug_logits(hsd_ctx *ctx, const void *workspace, int total_q, int n_seqs, float *logits,
                     void *cuda_stream);

/* Test-only: device address and size of a named intermediate of the last call (with that call's total_q
 * and n_seqs) inside `workspace`:
 * "x" fp32 [T,d_model] residual after the last layer, "h" bf16 [T,d_model] final-normed rows,
 * "q" bf16 [T,n_heads*head_dim], "attn" bf16 [T,n_heads*head_dim], "act" bf16 [T,d_ffn] of the last layer. */
HSD_API int hsd_debug_buffer(hsd_ctx *ctx, const void *workspace, int total_q, int n_seqs, const char *name,
                     void **ptr, size_t *bytes);

/* Test-only: arm a tap on an intermediate tensor of ONE decoder layer (Eq. 8 is a stack of such layers; the tap lets a
 * parity miss be traced to the layer where it starts).  The NEXT forward this context runs (hsd_prefill, hsd_verify_*)
 * copies, device to device on that call's stream and right after the kernel that produced it, the tensor `which` of
 * layer `layer` (0-based) into dst, then the tap disarms.  T = that call's packed rows.
 *   HSD_TAP_X       fp32 [T, d_model]            residual stream after the layer
 *   HSD_TAP_X_MID   fp32 [T, d_model]            residual stream after the layer's attention block
 *   HSD_TAP_H_ATTN  bf16 [T, d_model]            RMSNorm output that feeds the QKV projection
 *   HSD_TAP_H_FFN   bf16 [T, d_model]            RMSNorm output that feeds the gate/up projection
 *   HSD_TAP_Q       bf16 [T, n_heads*head_dim]   rotated queries
 *   HSD_TAP_ATTN    bf16 [T, n_heads*head_dim]   attention output
 *   HSD_TAP_ACT     bf16 [T, d_ffn]              SwiGLU activation
 *   dst             dev, dst_bytes bytes, caller-owned; a tensor larger than dst_bytes makes that forward return
 *                   HSD_ERR_WORKSPACE.  layer < 0 disarms.  Errors: INVALID_ARG (layer or which out of range, dst NULL). */
#define HSD_TAP_X 0
#define HSD_TAP_H_ATTN 1
#define HSD_TAP_H_FFN 2
#define HSD_TAP_Q 3
#define HSD_TAP_ATTN 4
#define HSD_TAP_ACT 5
#define HSD_TAP_X_MID 6
HSD_API int hsd_debug_tap(hsd_ctx *ctx, int layer, int which, void *dst, size_t dst_bytes);

/* Test/bench-only single operators, asynchronous on the stream.
 * hsd_op_linear: C = A W^T with the epilogue `mode`:
 *   0 store bf16 C[M,N]; 1 fp32 C[M,N] += result (residual add); 2 SwiGLU: W is [2N', K] (gate, up), writes
 *   bf16 C[M,N'] = silu(gate) * up with N = 2N' passed as n_out.
 *   A dev bf16 [M,K], W dev bf16 [n_out,K].  M >= 1; K, n_out multiples of 64. */
HSD_API int hsd_op_linear(hsd_ctx *ctx, const void *A, const void *W, void *C, int M, int n_out, int K, int mode,
                  void *cuda_stream);

/* Test-only: make hsd_op_linear use output tiles of `tile_n` columns (64, 128, 256, or 512 = a pair of CTAs sharing a
 * 256-row x 256-column tile) and, for mode 1, `k_slices`
 * slices of K per tile, instead of what the library would choose for the problem; 0 = choose.  A combination the
 * problem does not allow makes hsd_op_linear return HSD_ERR_CUDA.  Lets the parity tests reach every tile shape. */
HSD_API int hsd_debug_set_gemm_tile(hsd_ctx *ctx, int tile_n, int k_slices);

/* Test-only: the attention launch cuts the KV range of every query tile into slices so that it has about
 * `target_items` work items, none shorter than `min_kv_tiles` 128-token KV tiles (two paged blocks; 0 = the
 * library's defaults).
 * Results do not depend on the setting beyond fp32 summation order; tests use it to force many or no slices. */
HSD_API int hsd_debug_set_attn_plan(hsd_ctx *ctx, int target_items, int min_kv_tiles);

/* hsd_op_lm_head_argmax: the fused LM head on its own (Eq. 10 per row): for `rows` already-normalised hidden rows
 * h (dev bf16 [rows, d_model]) compute z = h W_lm^T tile by tile and keep only, per row, the argmax (lowest id on
 * ties), its logit, and the logit of next_tokens[row] (dev int32 [rows] or NULL; entries < 0 give NaN).  Logits
 * are never written to memory.
 *   scratch   dev, 8-byte aligned, at least rows * 8 bytes (the per-row running best), contents irrelevant
 *   argmax    dev int32 [rows] out;  zmax dev fp32 [rows] out;  zdraft dev fp32 [rows] out (required with
 *             next_tokens, else may be NULL)
 * Errors: INVALID_ARG, WORKSPACE (scratch too small / misaligned), CUDA. */
HSD_API int hsd_op_lm_head_argmax(hsd_ctx *ctx, const void *h, int rows, const int *next_tokens, void *scratch,
                          size_t scratch_bytes, int *argmax, float *zmax, float *zdraft, void *cuda_stream);

/* hsd_op_lm_head_argmax_noalloc: the same operator for callers that cannot allocate device memory.
 * (The paper has no counterpart; this is a packaging variant of the call above.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits, for example a plug-in called from inside another
 * framework's stream-ordered section, a real-time loop that must not take the allocator's lock, or a process
 * whose memory budget was handed out in full at start-up.  Such a caller already owns its inputs and outputs but
 * has nowhere to get the operator's scratch from, so the scratch is a fixed array inside the library instead:
 * HSD_NOALLOC_MAX_ROWS * 8 bytes (64 KB) of device memory that every GPU using the library holds until the
 * process exits.
 *
 *   h, rows, next_tokens, argmax, zmax, zdraft, cuda_stream: exactly as for hsd_op_lm_head_argmax.
 *   rows > HSD_NOALLOC_MAX_ROWS returns HSD_ERR_TOO_LONG and launches nothing.
 *   The context must belong to the current device (HSD_ERR_INVALID_ARG otherwise).
 *
 * The call makes no cudaMalloc / cudaFree and uses no allocating library routine.  The first call on each device
 * looks up the array's device address (one cudaGetSymbolAddress, checked); make that first call before any
 * stream capture starts, and from one thread.  All calls on a device share the one array: each call clears the
 * rows it uses before the GEMM, so nothing carries over from the previous call, but two calls whose kernels can
 * overlap on the GPU (different streams without an ordering between them) race on it and corrupt each other's
 * results.  Order them on one stream or with events. */
#define HSD_NOALLOC_MAX_ROWS 8192
HSD_API int hsd_op_lm_head_argmax_noalloc(hsd_ctx *ctx, const void *h, int rows, const int *next_tokens, int *argmax,
                                  float *zmax, float *zdraft, void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* HSD_H_ */
