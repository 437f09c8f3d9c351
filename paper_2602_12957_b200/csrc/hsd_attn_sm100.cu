// Varlen multi-query-token causal attention over the paged KV cache, tcgen05 / TMEM / TMA (sm_100a).
//
// A draft token attends to every committed row of its sequence and, causally, to the draft rows before it
// (the chain case of the paper's tree-ancestry mask, Sec. 3.2 / Fig. 2(c)).
//
// Work item = (q-tile, kv slice, kv head).  A q-tile is 128 MMA rows: 128/group consecutive tokens of one
// sequence x the `group` query heads that share the kv head (GQA packing, so K/V tiles are read once per
// group).  The KV range a q-tile can see is cut into up to kAttnMaxSplits slices so that a launch has about one item
// per CTA slot whatever the mix of context lengths (one page chunk over a long context, or many short regions); the
// plan is made once per step on the device (attn_plan_kernel) and reused by every layer.  Slices leave (unnormalised
// O, exponent reference, sum) partials in the workspace and the last slice to finish combines them in slice order, so
// the result does not depend on which CTA ran what.
//
// A KV tile is 128 keys = two paged blocks [64 keys][head_dim] per kv head, fetched by TMA through the block table,
// 64 dims at a time, into adjacent halves of a stage; K is the K-major B operand of S = Q K^T (one 128 x 128 x
// head_dim product per tile), V the MN-major B operand of O += P V (128 x head_dim x 128).  Persistent CTAs walk the
// item list: two per SM with head_dim 64, one with 128 (tensor-memory columns).  Warp roles:
// warp 0 = TMA producers (lane 0: Q and the K ring, lane 1: the V ring; K is free as soon as S has been formed, V
// only after the second product, so the two rings run at their own pace and two stages each suffice), warp 1 = MMA
// issuer + TMEM owner, warps 2..9 = softmax: warp w works on TMEM lane quarter w mod 4 (the hardware's rule), warps
// 2..5 on keys 0..63 of the tile and warps 6..9 on keys 64..127, one thread per (row, half).
// Per tile: S (TMEM, 128 fp32 columns) -> softmax in registers -> P (bf16, back into TMEM: 64 columns, the A operand
// of the second product, so P never passes through shared memory) -> O += P V accumulated in tensor memory.
// What the measurements behind this shape said (64-key tiles, four softmax warps, P through shared memory, per tile
// and CTA): the softmax warps' own instruction stream ~1,950 cycles, half of it the 64 exponentials of a row queueing
// with the other CTA's on the SM's 16 exp lanes per clock; the issuing thread ~1,300 (140-220 cycles for every probe
// of an already completed barrier, 70-90 per MMA or commit).  Twice the keys per barrier round and MMA group, twice
// the warps on the exponentials, and no shared-memory round trip for P attack both.
// The exponent reference of a row is not its running maximum but a value that is raised only when the maximum has
// grown by more than kRescaleBits binary orders since it was set (P stays below 2^kRescaleBits, far inside bf16 and
// fp32 range): then, and only then, the row's accumulator is read, scaled and written back; after the first tiles of
// a row that is rare.  The two threads of a row swap their halves' maxima through shared memory once per tile, so they
// take the same decisions.  Every wait is a bounded mbarrier wait, so one that gives up takes the whole CTA to the
// common exit.
#include "hsd_kernels.h"

namespace hsd {

constexpr int kSoftmaxWarps = 8;
constexpr int kAttnThreads = 32 * (2 + kSoftmaxWarps);
constexpr int KV_STAGES = 2;                       // per ring
constexpr int SUB_BYTES = 128 * 128;               // one K-major operand sub-tile: 128 rows (q rows / keys) x 64 dims
constexpr int KV_BLOCK_BYTES = 64 * 128;           // one paged block of K or of V for one kv head, 64 dims of it
constexpr int ATTN_BAR_BYTES = 256;
constexpr int ATTN_XCH_BYTES = 2 * 128 * 2 + 2 * 128 * 4;   // per (half, row): the tile's half-row maximum (bf16); the item's half-row sum (fp32)
constexpr float kRescaleBits = 8.f;
// Head dimension HD = 64 or 128.  An operand tile is HD / 64 sub-tiles of 64 dims each (a 128-byte-swizzled row is 64
// bf16): Q [sub][128 rows][64], a K or V stage [sub][block 0, block 1][64 keys][64].  The accumulator has HD columns.
// No alignment slack: with HD = 64 two CTAs of this size plus the per-CTA reserve share an SM, so the kernel relies
// on the 1024-byte alignment it declares for its dynamic shared memory (the swizzled tiles need it) and checks it.
template <int HD>
struct AttnCfg {
  static constexpr int NSUB = HD / 64;
  static constexpr int Q_BYTES = NSUB * SUB_BYTES;
  static constexpr int KV_TILE_BYTES = NSUB * SUB_BYTES;           // 128 keys
  static constexpr int SMEM = Q_BYTES + 2 * KV_STAGES * KV_TILE_BYTES + ATTN_XCH_BYTES + ATTN_BAR_BYTES;
  static constexpr int COL_O = 128, COL_P = 128 + HD;              // S: 128 fp32 columns, O: HD, P: 64 (two keys per column)
  static constexpr int TMEM_COLS = HD == 64 ? 256 : 512;           // allocations are powers of two
  static constexpr int CTAS_PER_SM = HD == 64 ? 2 : 1;             // tensor memory has 512 columns
  static constexpr int OWN = HD / 2;                               // accumulator columns of one softmax thread
};

struct AttnParams {
  AttnPlan plan;
  const int* block_table;
  int max_blocks, n_blocks, Hq, Hkv, group, layer;
  bf16* out;            // [T, Hq*HD]
  float* split_ws;      // partials of sliced items: [q-tile][kv head][slice][2 + HD][128 rows]
  const uint4* anc;     // [T] ancestry masks of candidate-tree rows, or nullptr: plain causal order within the call
  int* status;
};

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
  float y;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(y) : "f"(a), "f"(b), "f"(c));
  return y;
}
__device__ __forceinline__ void named_bar_sync(int id, int threads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}
// Barrier among whole warps on an mbarrier whose count is the number of warps: every lane's earlier shared-memory
// writes are visible to every participant afterwards.  `phase` counts this thread's uses of `bar`.
__device__ __forceinline__ bool warps_sync(uint64_t* bar, uint32_t& phase, int lane, volatile int* abort_flag,
                                           int* status, int where) {
  __syncwarp();
  if (lane == 0) mbar_arrive(bar);
  const bool ok = mbar_wait(bar, phase & 1u, abort_flag, status, where);
  ++phase;
  return __all_sync(0xffffffffu, ok);
}

// The item x kv-head index that CTA `bx` of a grid of `G` takes in round r of its walk (-1: none).  Round r: CTA i
// takes index r G + i in even rounds and r G + (G - 1 - i) in odd ones (the list is sorted longest first, so the CTA
// that drew a long item in one round draws a short one in the next).  A launch with fewer items than CTAs leaves
// some SMs with one busy CTA (the grid is two CTAs per SM, and CTA b shares its SM with CTA b + G/2 under the usual
// placement); a CTA that has its SM alone walks its tiles faster, so the longest items go to those SMs and the
// others pair a long item with a short one.
__device__ __forceinline__ int attn_item_at(int r, int total, int bx, int G) {
  const int n_rounds = (total + G - 1) / G, half_grid = G / 2;
  if (n_rounds == 1 && total > half_grid) {
    const int n_second = total - half_grid;            // busy CTAs in the second half of the grid
    if (bx < half_grid) return bx >= n_second ? bx - n_second : (half_grid - n_second) + bx;
    return bx - half_grid < n_second ? total - 1 - (bx - half_grid) : -1;
  }
  const int i = (r & 1) ? G - 1 - bx : bx;
  const int w = r * G + i;
  return w < total ? w : -1;
}

// ------------------------------------------------------------------------------------------------
// Plan: one CTA.  For every q-tile the KV tiles it can see and into how many slices that range is cut, then
// the flat list of (q-tile, slice) items with everything a CTA needs to run one.
__global__ void attn_plan_kernel(RowMeta rm, AttnPlan pl, KvView kv, int n_seqs, int tokens_per_tile, int target_items,
                                 int min_chunk, const int* tile_count, const int* status) {
  pdl_wait();
  pdl_launch_dependents();
  __shared__ int s_total;
  if (threadIdx.x == 0) s_total = 0;
  __syncthreads();
  if (*status) {
    if (threadIdx.x == 0) *pl.n_items = 0;
    for (int b = threadIdx.x; b < pl.grid; b += blockDim.x) pl.first[3 * b + 2] = make_int4(-1, 0, 0, 0);
    return;
  }
  const int n_tiles = *tile_count;
  int my = 0;
  for (int s = threadIdx.x; s < n_seqs; s += blockDim.x) {
    const int t0 = rm.seq_tile0[s], t1 = rm.seq_tile0[s + 1];
    const int L = rm.seq_len[s], n = rm.seq_n[s];
    for (int t = t0; t < t1; ++t) {
      const int tok_end = min(n, (t - t0 + 1) * tokens_per_tile);
      const int n_kv = (L + tok_end + 127) >> 7;         // 128-key tiles (two paged blocks): the unit slices are cut in
      pl.tile_seq[t] = s;
      pl.tile_nkv[t] = n_kv;
      my += n_kv;
    }
  }
  atomicAdd(&s_total, my);
  __syncthreads();
  // KV tiles per slice: start from an even share.  Rounding up the slice count of every q-tile can leave the
  // launch with somewhat more items than CTA slots, and then the few CTAs that draw a second item double its
  // length: in that band (1 to 1.6 items per slot) the share is grown until every slot has at most one item.
  // Well beyond it a second round is about full and the sorted walk balances it, so the share is kept.
  __shared__ int s_n, s_count, s_longest;
  int chunk = max(min_chunk, (s_total + target_items - 1) / max(1, target_items));
  for (int it = 0; it < 256; ++it) {                      // every thread runs the same iterations
    if (threadIdx.x == 0) { s_count = 0; s_longest = 0; }
    __syncthreads();
    int count = 0, longest = 0;
    for (int t = threadIdx.x; t < n_tiles; t += blockDim.x) {
      const int n_kv = pl.tile_nkv[t];
      count += max(1, min(kAttnMaxSplits, (n_kv + chunk - 1) / chunk));
      longest = max(longest, n_kv);
    }
    atomicAdd(&s_count, count);
    atomicMax(&s_longest, longest);
    __syncthreads();
    const bool done = s_count <= target_items || 5 * s_count >= 8 * target_items || chunk >= s_longest;
    __syncthreads();
    if (done) break;
    chunk += max(1, chunk >> 4);
  }
  if (threadIdx.x == 0) {
    int n = 0;
    for (int t = 0; t < n_tiles; ++t) {   // serial: a few hundred tiles at most, once per step
      const int n_kv = pl.tile_nkv[t];
      const int s = pl.tile_seq[t];
      const int tok0 = (t - rm.seq_tile0[s]) * tokens_per_tile;
      const int n_tok = min(tokens_per_tile, rm.seq_n[s] - tok0);
      const int blocks = (rm.seq_len[s] + tok0 + n_tok + 63) >> 6;    // 64-key blocks the q-tile can see
      const int ns = max(1, min(kAttnMaxSplits, (n_kv + chunk - 1) / chunk));
      const int base = n_kv / ns, rem = n_kv % ns;
      int lo = 0;
      for (int k = 0; k < ns; ++k) {
        const int len = base + (k < rem ? 1 : 0);
        // the item's range in 64-key blocks: only the last slice of a q-tile can end on half a tile
        pl.items_unsorted[2 * n] = make_int4(rm.seq_q0[s] + tok0, rm.seq_len[s] + tok0, n_tok, rm.seq_slot[s]);
        pl.items_unsorted[2 * n + 1] = make_int4((2 * lo) | (min(blocks, 2 * (lo + len)) << 16), k | (ns << 8) | (tok0 << 16), t, len);
        ++n;
        lo += len;
      }
    }
    *pl.n_items = n;
    s_n = n;
  }
  __syncthreads();
  // longest first (rank sort, ties by creation order): the attention CTAs walk the list in boustrophedon order, so
  // every CTA's share of KV tiles comes out about equal
  const int n = s_n;
  for (int i = threadIdx.x; i < n; i += blockDim.x) {
    const int len = pl.items_unsorted[2 * i + 1].w;
    int rank = 0;
    for (int k = 0; k < n; ++k) {
      const int lk = pl.items_unsorted[2 * k + 1].w;
      rank += (lk > len) || (lk == len && k < i);
    }
    pl.items[2 * rank] = pl.items_unsorted[2 * i];
    pl.items[2 * rank + 1] = pl.items_unsorted[2 * i + 1];
  }
  // slice-arrival counters of every (q-tile, kv head): zero at the start of a step, reset by the combiner
  for (int i = threadIdx.x; i < n_tiles * pl.n_kv_heads; i += blockDim.x) pl.counters[i] = 0;
  // what every CTA of the attention grid starts with, in one record: its first item and the physical blocks of that
  // item's first KV tile, so that a CTA's first loads do not wait for a chain of dependent reads (item -> block table)
  __syncthreads();
  const int total = n * pl.n_kv_heads;
  for (int b = threadIdx.x; b < pl.grid; b += blockDim.x) {
    const int w = attn_item_at(0, total, b, pl.grid);
    if (w < 0) {
      pl.first[3 * b + 2] = make_int4(-1, 0, 0, 0);
      continue;
    }
    const int4 ia = pl.items[2 * (w / pl.n_kv_heads)], ib = pl.items[2 * (w / pl.n_kv_heads) + 1];
    const int kt_lo = ib.x & 0xffff, kt_hi = ib.x >> 16;
    int phys0 = 0, phys1 = 0;
    if (kt_hi > kt_lo && ia.w >= 0 && ia.w < kv.n_slots && kt_hi <= kv.max_blocks) {
      const int* bt = kv.block_table + (size_t)ia.w * kv.max_blocks;
      phys0 = bt[kt_lo];
      phys1 = bt[kt_lo + 1 < kt_hi ? kt_lo + 1 : kt_lo];
    }
    pl.first[3 * b] = ia;
    pl.first[3 * b + 1] = ib;
    pl.first[3 * b + 2] = make_int4(w, w % pl.n_kv_heads, phys0, phys1);
  }
}

void launch_attn_plan(cudaStream_t st, const RowMeta& rm, const AttnPlan& pl, const KvView& kv, int n_seqs,
                      int tokens_per_tile, int target_items, int min_chunk, const int* tile_count, const int* status,
                      bool pdl) {
  launch_kernel(attn_plan_kernel, dim3(1), dim3(256), 0, st, pdl, rm, pl, kv, n_seqs, tokens_per_tile, target_items,
                min_chunk, tile_count, status);
}

// ------------------------------------------------------------------------------------------------
template <int HD>
__global__ void __launch_bounds__(kAttnThreads, AttnCfg<HD>::CTAS_PER_SM)
attn_sm100_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                  const __grid_constant__ CUtensorMap tmV, AttnParams p) {
  using C = AttnCfg<HD>;
  constexpr int Q_BYTES = C::Q_BYTES, KV_TILE_BYTES = C::KV_TILE_BYTES, NSUB = C::NSUB;
  constexpr int TMEM_COL_O = C::COL_O, TMEM_COL_P = C::COL_P, OWN = C::OWN;
  extern __shared__ __align__(1024) uint8_t smem[];
  uint8_t* sQ = smem;
  uint8_t* sK = sQ + Q_BYTES;                          // ring stage s: sK + s * KV_TILE_BYTES, per sub-tile block 0 then block 1
  uint8_t* sV = sK + KV_STAGES * KV_TILE_BYTES;
  __nv_bfloat16* xch = reinterpret_cast<__nv_bfloat16*>(sV + KV_STAGES * KV_TILE_BYTES);   // [half][row] maxima
  float* lx = reinterpret_cast<float*>(xch + 2 * 128);                                         // [half][row] sums
  uint64_t* bars = reinterpret_cast<uint64_t*>(sV + KV_STAGES * KV_TILE_BYTES + ATTN_XCH_BYTES);
  uint64_t* q_full = bars;                 // Q tile landed                       (one phase per item)
  uint64_t* q_empty = bars + 1;            // every S MMA of the item has read Q   (one phase per item)
  uint64_t* k_full = bars + 2;             // [stage]
  uint64_t* k_empty = k_full + KV_STAGES;  // [stage] S of the tile has been formed
  uint64_t* v_full = k_empty + KV_STAGES;
  uint64_t* v_empty = v_full + KV_STAGES;  // [stage] O += P V of the tile has completed
  uint64_t* s_full = v_empty + KV_STAGES;  // S(t) is in tensor memory
  uint64_t* s_empty = s_full + 1;          // the softmax warps hold S(t) in registers
  uint64_t* p_full = s_empty + 1;          // P(t) is in tensor memory (and the accumulator rescaled, if it had to be)
  uint64_t* o_full = p_full + 1;           // O += P(t) V(t) has completed
  uint64_t* group_bar = o_full + 1;        // the eight softmax warps (slice hand-over)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(group_bar + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  volatile int* s_flag = abort_flag + 1;   // combine: "this CTA ran the last slice to finish"

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (smem_u32(smem) & 1023u) {            // uniform over the CTA: nothing has been set up yet
    if (threadIdx.x == 0) dev_fail(p.status, DEV_WAIT_TIMEOUT, 499);
    return;
  }
  if (threadIdx.x == 0) {
    mbar_init(q_full, 1);
    mbar_init(q_empty, 1);
    for (int s = 0; s < KV_STAGES; ++s) {
      mbar_init(k_full + s, 1);
      mbar_init(k_empty + s, 1);
      mbar_init(v_full + s, 1);
      mbar_init(v_empty + s, 1);
    }
    mbar_init(s_full, 1);
    mbar_init(s_empty, kSoftmaxWarps);
    mbar_init(p_full, kSoftmaxWarps);
    mbar_init(o_full, 1);
    mbar_init(group_bar, kSoftmaxWarps);
    *abort_flag = 0;
    fence_mbar_init();
    tma_prefetch_desc(&tmQ);
    tma_prefetch_desc(&tmK);
    tma_prefetch_desc(&tmV);
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, C::TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  pdl_wait();               // q, the K/V rows of this step, the row metadata and the plan come from earlier kernels
  pdl_launch_dependents();

  // The plan's record of this CTA's first item (the item and the physical blocks of its first KV tile) for the two
  // warps that start the pipeline: read together with the status word and the item count, before any of them is
  // used, so that the first TMA loads are one round trip away instead of four (status -> count -> item -> block table).
  int4 rec_a = make_int4(0, 0, 0, 0), rec_b = rec_a, rec_c = rec_a;
  if (warp < 2) {
    const int4* rec = p.plan.first + 3 * (size_t)blockIdx.x;
    rec_a = rec[0];
    rec_b = rec[1];
    rec_c = rec[2];
  }
  const int status_now = *p.status, n_items_now = *p.plan.n_items;
  const int total = status_now ? 0 : n_items_now * p.Hkv;
  const int n_rounds = (total + (int)gridDim.x - 1) / (int)gridDim.x;
  auto item_of_round = [&](int r) -> int { return attn_item_at(r, total, (int)blockIdx.x, (int)gridDim.x); };

  // Tile counter t (all 128-key tiles of all items of this CTA): ring stage = t % KV_STAGES, and every barrier's
  // parity follows from how often t has used it; n counts items (Q hand-over barriers).
  if (warp == 0) {
    if (lane < 2) {
      // lane 0: Q and the K ring; lane 1: the V ring
      const bool is_k = lane == 0;
      uint64_t* full = is_k ? k_full : v_full;
      uint64_t* empty = is_k ? k_empty : v_empty;
      uint8_t* ring = is_k ? sK : sV;
      const CUtensorMap* tm = is_k ? &tmK : &tmV;
      uint32_t t = 0;
      int n = 0;
      for (int r = 0; r < n_rounds; ++r) {
        const int w = r == 0 ? (total > 0 ? rec_c.x : -1) : item_of_round(r);
        if (w < 0) continue;
        int4 ia = rec_a, ib = rec_b;
        int kvh = rec_c.y;
        if (r != 0) {
          ia = p.plan.items[2 * (w / p.Hkv)];
          ib = p.plan.items[2 * (w / p.Hkv) + 1];
          kvh = w % p.Hkv;
        }
        const int kt_lo = ib.x & 0xffff, kt_hi = ib.x >> 16;
        const int* bt = p.block_table + (size_t)ia.w * p.max_blocks;
        if (is_k) {
          if (!mbar_wait(q_empty, (n & 1) ^ 1u, abort_flag, p.status, 400)) goto done;
          mbar_expect_tx(q_full, Q_BYTES);
#pragma unroll
          for (int h = 0; h < NSUB; ++h) tma_load_3d(sQ + h * SUB_BYTES, &tmQ, q_full, 64 * h, kvh * p.group, ia.x);
        }
        for (int kt = kt_lo; kt < kt_hi; kt += 2, ++t) {
          // the tile's two blocks; a slice of odd length ends with half a tile: the last block is staged twice and
          // the softmax warps mask its second copy
          int phys0 = rec_c.z, phys1 = rec_c.w;
          if (r != 0 || kt != kt_lo) {
            phys0 = bt[kt];
            phys1 = bt[kt + 1 < kt_hi ? kt + 1 : kt];
          }
          const int st = t % KV_STAGES;
          if (!mbar_wait(empty + st, ((t / KV_STAGES) & 1) ^ 1u, abort_flag, p.status, 401)) goto done;
          const int row0 = (((p.layer * p.n_blocks) + phys0) * p.Hkv + kvh) * 64;
          const int row1 = (((p.layer * p.n_blocks) + phys1) * p.Hkv + kvh) * 64;
          uint8_t* dst = ring + st * KV_TILE_BYTES;
          mbar_expect_tx(full + st, KV_TILE_BYTES);
#pragma unroll
          for (int h = 0; h < NSUB; ++h) {
            tma_load_2d(dst + h * SUB_BYTES, tm, full + st, 64 * h, row0);
            tma_load_2d(dst + h * SUB_BYTES + KV_BLOCK_BYTES, tm, full + st, 64 * h, row1);
          }
        }
        ++n;
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc_s = umma_idesc_bf16(128);
      constexpr uint32_t idesc_pv = umma_idesc_bf16(64, true);
      const uint32_t q_addr = smem_u32(sQ);
      uint32_t t = 0;
      int n = 0;
      for (int r = 0; r < n_rounds; ++r) {
        const int w = r == 0 ? (total > 0 ? rec_c.x : -1) : item_of_round(r);
        if (w < 0) continue;
        const int4 ib = r == 0 ? rec_b : p.plan.items[2 * (w / p.Hkv) + 1];
        const int n_it = ((ib.x >> 16) - (ib.x & 0xffff) + 1) / 2;      // 128-key tiles of the item
        // S(ti) = Q K(ti)^T: four K = 16 steps over every 64 dims, N = 128 keys
        auto issue_s = [&](uint32_t ti, bool last) -> bool {
          const int st = ti % KV_STAGES;
          if (!mbar_wait(k_full + st, (ti / KV_STAGES) & 1, abort_flag, p.status, 410)) return false;
          if (!mbar_wait(s_empty, (ti & 1) ^ 1u, abort_flag, p.status, 411)) return false;   // S(ti - 1) is in registers
          tc_fence_after();
          const uint32_t k_addr = smem_u32(sK + st * KV_TILE_BYTES);
#pragma unroll
          for (int h = 0; h < NSUB; ++h)
#pragma unroll
            for (int k = 0; k < 4; ++k)
              umma_bf16(tmem_base, umma_desc_sw128(q_addr + h * SUB_BYTES + k * 32),
                        umma_desc_sw128(k_addr + h * SUB_BYTES + k * 32), idesc_s, (h | k) != 0);
          umma_commit(s_full);
          umma_commit(k_empty + st);              // K is free once S has been formed
          if (last) umma_commit(q_empty);         // last S MMA of the item: Q is free once it completes
          return true;
        };
        if (!mbar_wait(q_full, n & 1, abort_flag, p.status, 412)) goto done;
        if (!issue_s(t, n_it == 1)) goto done;
        for (int j = 0; j < n_it; ++j, ++t) {
          if (j + 1 < n_it && !issue_s(t + 1, j + 2 == n_it)) goto done;
          // P(t) is written, and whatever had to be done to the accumulator before this product is done
          if (!mbar_wait(p_full, t & 1, abort_flag, p.status, 413)) goto done;
          const int st = t % KV_STAGES;
          if (!mbar_wait(v_full + st, (t / KV_STAGES) & 1, abort_flag, p.status, 415)) goto done;
          tc_fence_after();
          const uint32_t v_addr = smem_u32(sV + st * KV_TILE_BYTES);
          const uint32_t d = tmem_base + TMEM_COL_O;   // the item's accumulator: the first product of an item overwrites it
#pragma unroll
          for (int h = 0; h < NSUB; ++h)   // 64 output dims per product
#pragma unroll
            for (int k = 0; k < 8; ++k)    // 16 keys per step: 8 columns of P in tensor memory; V [key][dim] is MN-major,
                                           // a step of 16 keys is 16 rows of 128 bytes
              umma_bf16_ta(d + 64 * h, tmem_base + TMEM_COL_P + k * 8, umma_desc_sw128(v_addr + h * SUB_BYTES + k * 2048),
                           idesc_pv, (j != 0 || k != 0) ? 1u : 0u);
          umma_commit(v_empty + st);
          umma_commit(o_full);
        }
        ++n;
      }
      // every stage-release arrival must land before the CTA's shared memory can be handed on
      if (t > 0 && !mbar_wait(o_full, (t - 1) & 1, abort_flag, p.status, 414)) goto done;
    }
  } else {
    const int quarter = warp & 3;                      // TMEM lane quarter a warp may touch = warp id mod 4
    const int half = (warp - 2) >> 2;                  // keys [64 half, 64 half + 64) of every tile
    const int row = quarter * 32 + lane;               // q row of the tile = TMEM lane
    const int tok = row / p.group;
    const uint32_t t_lane = tmem_base + (uint32_t(quarter * 32) << 16);
    const uint32_t t_o = t_lane + TMEM_COL_O + half * OWN;    // this thread's OWN columns of the accumulator row
    const uint32_t t_p = t_lane + TMEM_COL_P + half * 32;     // and of the row of P: its 64 keys, two per column
    const float sc = (HD == 64 ? 0.125f : 0.08838834764831845f) * 1.4426950408889634f;     // 1/sqrt(HD) * log2(e)
    uint32_t t = 0, group_ph = 0;
    for (int r = 0; r < n_rounds; ++r) {
      const int w = item_of_round(r);
      if (w < 0) continue;
      const int4 ia = p.plan.items[2 * (w / p.Hkv)], ib = p.plan.items[2 * (w / p.Hkv) + 1];
      const int kvh = w % p.Hkv;
      const int q_row0 = ia.x, pos0 = ia.y, n_tok = ia.z;
      const int kt_lo = ib.x & 0xffff, kt_hi = ib.x >> 16;
      const int split = ib.y & 0xff, n_split = (ib.y >> 8) & 0xff;
      const int pos_row = pos0 + tok;
      const bool row_ok = tok < n_tok;
      // candidate trees (Sec. 3.2, Fig. 2(c)): a row sees the committed context and, of the rows of this call, only
      // itself and its ancestors.  len0 = committed length; the mask's bit i stands for cache row len0 + i.
      const int len0 = pos0 - (ib.y >> 16);
      uint4 am = make_uint4(0u, 0u, 0u, 0u);
      if (p.anc && row_ok) am = p.anc[q_row0 + tok];
      // warp-uniform: some row of this warp is a real token.  A ragged last q-tile leaves whole warps without one;
      // they keep step with the barriers but skip the loads, the exps and the P rows (which only feed their own,
      // never stored, output rows)
      const bool warp_ok = (quarter * 32) / p.group < n_tok;
      float m_ref = -INFINITY, l = 0.f;                // exponent reference (log2 units, scaled); sum of this thread's P
      // visibility of the 32 keys from `key0` on for this thread's row, as a bit mask
      auto visible = [&](int key0, int key_end) -> uint32_t {
        if (key0 >= key_end) return 0u;                 // the second copy of a slice's last block
        if (p.anc) {
          auto word = [&](int i) -> uint32_t {
            return i < 0 ? 0xffffffffu : i == 0 ? am.x : i == 1 ? am.y : i == 2 ? am.z : i == 3 ? am.w : 0u;
          };
          const int pos = key0 - len0;
          if (pos <= -32) return 0xffffffffu;
          if (pos >= 128) return 0u;
          const int wi = pos >> 5;                      // floor, also for negative positions
          return __funnelshift_r(word(wi), word(wi + 1), pos & 31);
        }
        const int nvis = pos_row - key0 + 1;            // keys key0 .. pos_row are visible
        return nvis >= 32 ? 0xffffffffu : (nvis <= 0 ? 0u : ((1u << nvis) - 1u));
      };

      for (int kt = kt_lo; kt < kt_hi; kt += 2, ++t) {
        bool ok = mbar_wait(s_full, t & 1, abort_flag, p.status, 420);
        if (!__all_sync(0xffffffffu, ok)) goto done;
        tc_fence_after();
        if (!warp_ok) {
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(s_empty);
          // S(t + 1) is issued before P(t) is consumed, so this warp could be back here for the next tile while phase
          // t of p_full is still open, and its arrival would then be counted there: like the warps that do write P,
          // it arrives for tile t only once the product of tile t - 1 (hence phase t - 1 of p_full) is complete
          if (t > 0) {
            ok = mbar_wait(o_full, (t - 1) & 1, abort_flag, p.status, 424);
            if (!__all_sync(0xffffffffu, ok)) goto done;
          }
          if (lane == 0) mbar_arrive(p_full);
          continue;
        }
        const int key_end = min(kt + 2, kt_hi) * 64;    // keys of this tile that belong to the slice
        const int kb_own = kt * 64 + half * 64;
        // does any key of the tile need masking for some row of the q-tile?  (warp-uniform)
        const bool masked_tile = p.anc ? (kt * 64 + 127 >= len0) : (kt * 64 + 127 > pos0);
        const bool partial_tile = key_end < kt * 64 + 128;
        uint32_t s0[32], s1[32];
        tmem_ld32(t_lane + half * 64, s0);
        tmem_ld32(t_lane + half * 64 + 32, s1);
        tmem_ld_wait();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(s_empty);
        if (masked_tile || partial_tile) {
          const uint32_t v0 = visible(kb_own, key_end), v1 = visible(kb_own + 32, key_end);
#pragma unroll
          for (int e = 0; e < 32; ++e) {
            if (!((v0 >> e) & 1u)) s0[e] = 0xff800000u;            // -inf
            if (!((v1 >> e) & 1u)) s1[e] = 0xff800000u;
          }
        }
        float mx = -INFINITY, mx_b = -INFINITY;              // two chains
#pragma unroll
        for (int e = 0; e < 32; e += 2) {
          mx = max3(mx, __uint_as_float(s0[e]), __uint_as_float(s1[e]));
          mx_b = max3(mx_b, __uint_as_float(s0[e + 1]), __uint_as_float(s1[e + 1]));
        }
        mx = fmaxf(mx, mx_b);
        // The row's maximum over all 128 keys: the two threads of a row swap their halves' maxima through shared memory.
        // Both use the bf16-rounded values of BOTH halves, so they arrive at the same number (the reference only has to
        // be near the maximum, and identical for the row's two threads).
        {
          const __nv_bfloat16 mine = __float2bfloat16_rn(mx);
          xch[half * 128 + row] = mine;
          named_bar_sync(1 + quarter, 64);                 // the two warps of this lane quarter
          mx = fmaxf(__bfloat162float(mine), __bfloat162float(xch[(half ^ 1) * 128 + row]));
          named_bar_sync(1 + quarter, 64);                 // both have read before either writes the next tile's
        }
        mx *= sc;
        // The reference moves only when the maximum has outgrown it by more than kRescaleBits (or nothing has been
        // accumulated under it yet: then moving it costs nothing).  `l` is this thread's half of the row sum; whether
        // anything has been accumulated is a property of the row, so the test uses the reference itself.
        float alpha = 1.f;
        bool rescale = false;
        if (mx > m_ref) {
          if (m_ref == -INFINITY) {
            m_ref = mx;                                   // nothing accumulated so far (first tile, or all keys masked)
          } else if (mx > m_ref + kRescaleBits) {
            alpha = ex2(m_ref - mx);
            m_ref = mx;
            rescale = true;
          }
        }
        const float m_use = (m_ref == -INFINITY) ? 0.f : m_ref;
        float sum = 0.f, sum_b = 0.f, sum_c = 0.f, sum_d = 0.f;   // four chains
        uint32_t pk[32];
#pragma unroll
        for (int e = 0; e < 16; ++e) {
          const float a0 = ex2(fmaf(__uint_as_float(s0[2 * e]), sc, -m_use));
          const float a1 = ex2(fmaf(__uint_as_float(s0[2 * e + 1]), sc, -m_use));
          if (e & 1) sum_b += a0 + a1; else sum += a0 + a1;
          pk[e] = pack_bf16(a0, a1);
        }
#pragma unroll
        for (int e = 0; e < 16; ++e) {
          const float a0 = ex2(fmaf(__uint_as_float(s1[2 * e]), sc, -m_use));
          const float a1 = ex2(fmaf(__uint_as_float(s1[2 * e + 1]), sc, -m_use));
          if (e & 1) sum_d += a0 + a1; else sum_c += a0 + a1;
          pk[16 + e] = pack_bf16(a0, a1);
        }
        l = l * alpha + ((sum + sum_b) + (sum_c + sum_d));
        // P's columns are read by the product of tile t - 1, which also still adds into the accumulator
        if (t > 0) {
          ok = mbar_wait(o_full, (t - 1) & 1, abort_flag, p.status, 421);
          if (!__all_sync(0xffffffffu, ok)) goto done;
          tc_fence_after();
        }
        if (__any_sync(0xffffffffu, rescale)) {
          // rare: scale this thread's half of the accumulator row (alpha = 1 where not needed)
#pragma unroll 1
          for (int c = 0; c < OWN; c += 32) {
            uint32_t o[32];
            tmem_ld32(t_o + c, o);
            tmem_ld_wait();
#pragma unroll
            for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
            tmem_st32(t_o + c, o);
          }
          tmem_st_wait();
          tc_fence_before();
        }
        // P row -> tensor memory, where the second product reads it as its A operand (no shared-memory round trip)
        tmem_st32(t_p, pk);
        tmem_st_wait();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(p_full);
      }
      // the item's last product (products complete in issue order, so all of them)
      if (kt_hi > kt_lo) {
        bool ok = mbar_wait(o_full, (t - 1) & 1, abort_flag, p.status, 422);
        if (!__all_sync(0xffffffffu, ok)) goto done;
        tc_fence_after();
      }
      // the row sum is the sum of its two threads' halves
      float l_row = l;
      if (warp_ok) {
        lx[half * 128 + row] = l;
        named_bar_sync(1 + quarter, 64);                 // the two warps of this lane quarter
        l_row += lx[(half ^ 1) * 128 + row];
        named_bar_sync(1 + quarter, 64);                 // both have read before either writes the next item's
      }

      // ---- item epilogue: this thread owns dims [OWN half, OWN half + OWN) of its row
      const int head = kvh * p.group + row % p.group;
      uint4* out_row = reinterpret_cast<uint4*>(p.out + (size_t)(q_row0 + tok) * p.Hq * HD + head * HD + half * OWN);
      if (n_split == 1) {
        if (warp_ok) {                                     // (a whole warp reads tensor memory together)
          const float inv = 1.f / l_row;
#pragma unroll 1
          for (int c0 = 0; c0 < OWN; c0 += 32) {
            uint32_t o[32];
            tmem_ld32(t_o + c0, o);
            tmem_ld_wait();
            if (row_ok) {
              uint4* dst = out_row + c0 / 8;
#pragma unroll
              for (int c = 0; c < 4; ++c)
                dst[c] = make_uint4(
                    pack_bf16(__uint_as_float(o[8 * c]) * inv, __uint_as_float(o[8 * c + 1]) * inv),
                    pack_bf16(__uint_as_float(o[8 * c + 2]) * inv, __uint_as_float(o[8 * c + 3]) * inv),
                    pack_bf16(__uint_as_float(o[8 * c + 4]) * inv, __uint_as_float(o[8 * c + 5]) * inv),
                    pack_bf16(__uint_as_float(o[8 * c + 6]) * inv, __uint_as_float(o[8 * c + 7]) * inv));
            }
          }
          tc_fence_before();
        }
      } else {
        // partials of this (q-tile, kv head): [slice][2 + HD][128 rows] floats, entry 0 the exponent reference (log2
        // units), 1 the row sum under it, 2.. the HD unnormalised outputs; a warp's accesses are 128-byte lines
        constexpr int PART = (2 + HD) * 128;
        float* tile_part = p.split_ws + ((size_t)(ib.z * p.Hkv + kvh) * kAttnMaxSplits) * PART + row;
        if (warp_ok) {
          float* part = tile_part + (size_t)split * PART;
          if (half == 0) {
            part[0] = m_ref;
            part[128] = l_row;
          }
#pragma unroll 1
          for (int c0 = 0; c0 < OWN; c0 += 32) {
            uint32_t o[32];
            tmem_ld32(t_o + c0, o);
            tmem_ld_wait();
#pragma unroll
            for (int e = 0; e < 32; ++e) part[(2 + half * OWN + c0 + e) * 128] = __uint_as_float(o[e]);
          }
          tc_fence_before();
        }
        __threadfence();
        if (!warps_sync(group_bar, group_ph, lane, abort_flag, p.status, 427)) goto done;
        if (warp == 2 && lane == 0) {
          int* ctr = p.plan.counters + ib.z * p.Hkv + kvh;
          const int old = atomicAdd(ctr, 1);
          *s_flag = (old == n_split - 1);
          if (old == n_split - 1) *ctr = 0;             // ready for the next layer
        }
        if (!warps_sync(group_bar, group_ph, lane, abort_flag, p.status, 428)) goto done;
        if (*s_flag && warp_ok) {
          __threadfence();
          float M = -INFINITY;
          for (int s = 0; s < n_split; ++s) M = fmaxf(M, __ldcg(tile_part + (size_t)s * PART));
#pragma unroll 1
          for (int c0 = 0; c0 < OWN; c0 += 32) {
            float Lsum = 0.f;
            float o[32];
#pragma unroll
            for (int e = 0; e < 32; ++e) o[e] = 0.f;
            for (int s = 0; s < n_split; ++s) {           // fixed slice order: the result does not depend on arrival
              const float* ps = tile_part + (size_t)s * PART;
              const float mxs = __ldcg(ps);
              const float wgt = (mxs == -INFINITY) ? 0.f : ex2(mxs - M);
              Lsum += wgt * __ldcg(ps + 128);
#pragma unroll
              for (int e = 0; e < 32; ++e) o[e] += wgt * __ldcg(ps + (2 + half * OWN + c0 + e) * 128);
            }
            if (row_ok) {
              const float inv = 1.f / Lsum;
              uint4* dst = out_row + c0 / 8;
#pragma unroll
              for (int c = 0; c < 4; ++c)
                dst[c] = make_uint4(pack_bf16(o[8 * c] * inv, o[8 * c + 1] * inv), pack_bf16(o[8 * c + 2] * inv, o[8 * c + 3] * inv),
                                    pack_bf16(o[8 * c + 4] * inv, o[8 * c + 5] * inv), pack_bf16(o[8 * c + 6] * inv, o[8 * c + 7] * inv));
            }
          }
        }
        // s_flag is rewritten by the next item only after all have read it
        if (!warps_sync(group_bar, group_ph, lane, abort_flag, p.status, 429)) goto done;
      }
    }
  }

done:
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    if (*abort_flag) __nanosleep(20000);
    tmem_dealloc(tmem_base, C::TMEM_COLS);
  }
}

int launch_attn_sm100(cudaStream_t st, const CUtensorMap& tmQ, const CUtensorMap& tmK, const CUtensorMap& tmV,
                      const AttnPlan& plan, const KvView& kv, const ModelDims& md, int layer, bf16* out, int n_sms,
                      int device, int* status, float* split_ws, const uint4* anc, bool pdl) {
  static bool attr_set[2][kMaxDevices] = {};       // the attribute is per kernel and device
  if (device < 0 || device >= kMaxDevices || (md.D != 64 && md.D != 128)) return -1;
  const int which = md.D == 128;
  if (!attr_set[which][device]) {
    const cudaError_t e =
        which ? cudaFuncSetAttribute(attn_sm100_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, AttnCfg<128>::SMEM)
              : cudaFuncSetAttribute(attn_sm100_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, AttnCfg<64>::SMEM);
    if (e != cudaSuccess) return -1;
    attr_set[which][device] = true;
  }
  AttnParams p;
  p.plan = plan;
  p.block_table = kv.block_table;
  p.max_blocks = kv.max_blocks;
  p.n_blocks = kv.n_blocks;
  p.Hq = md.Hq;
  p.Hkv = md.Hkv;
  p.group = md.group;
  p.layer = layer;
  p.out = out;
  p.split_ws = split_ws;
  p.anc = anc;
  p.status = status;
  if (which)
    return launch_kernel(attn_sm100_kernel<128>, dim3(plan.grid), dim3(kAttnThreads), AttnCfg<128>::SMEM, st, pdl, tmQ, tmK,
                         tmV, p);
  return launch_kernel(attn_sm100_kernel<64>, dim3(plan.grid), dim3(kAttnThreads), AttnCfg<64>::SMEM, st, pdl, tmQ, tmK, tmV, p);
}

}  // namespace hsd
