// Varlen multi-query-token causal attention over the paged KV cache, tcgen05 / TMEM / TMA (sm_100a).
//
// A draft token attends to every committed row of its sequence and, causally, to the draft rows before it
// (the chain case of the paper's tree-ancestry mask, Sec. 3.2 / Fig. 2(c)).
//
// Work item = (q-tile, kv slice, kv head).  A q-tile is 128 MMA rows: 128/group consecutive tokens of one
// sequence x the `group` query heads that share the kv head (GQA packing, so K/V tiles are read once per
// group).  K and V tiles [64 keys][64 dims] are exactly one paged block per kv head, fetched by TMA through
// the block table; K is the K-major B operand of S = Q K^T, V the MN-major B operand of P V.  The KV range a q-tile can see is cut into up to
// kAttnMaxSplits slices so that a launch has a few items per CTA slot whatever the mix of context lengths
// (one page chunk over a long context, or many short regions); the plan is made once per step on the
// device (attn_plan_kernel) and reused by every layer.  Slices leave (unnormalised O, max, sum) partials in
// the workspace and the last slice to finish combines them in slice order, so the result does not depend
// on which CTA ran what.
//
// Persistent CTAs, two per SM, walk the item list.  Warp roles: warp 0 = TMA producer, warp 1 = MMA issuer +
// TMEM owner, warps 2..5 = softmax (one TMEM lane quarter each, one thread per q row, no shuffles).
// Per KV tile: S = Q K^T (TMEM) -> softmax in registers -> P (bf16, shared memory, 128B-swizzled) -> O += P V,
// accumulated IN TENSOR MEMORY.  S and P are double-buffered, so the tensor pipe works on tile j+1 while the softmax
// warps are on tile j, and a softmax warp never waits for a product younger than the one two tiles back: measured with
// every arithmetic instruction removed, a loop in which each tile waits for the product of the tile before it still
// took four fifths of the kernel's time (two barrier hand-overs per tile on the critical path); with the accumulator
// in tensor memory nothing in the steady state waits on a hand-over at all.  The exponent reference of a row is not
// its running maximum but a value that is raised only when the maximum has grown by more than kRescaleBits binary
// orders since it was set (P stays below 2^kRescaleBits, far inside bf16 and fp32 range): then, and only then, the
// row's accumulator is read, scaled and written back.  After the first tiles of a row that is rare.  Two CTAs per SM
// interleave further.  Every wait is a bounded mbarrier wait, so one that gives up takes the whole CTA to the common exit.
#include "hsd_kernels.h"

namespace hsd {

constexpr int kAttnThreads = 192;
constexpr int KV_STAGES = 3;
constexpr int Q_BYTES = 128 * 128;
constexpr int KV_TILE_BYTES = 64 * 128;            // one K tile or one V tile
constexpr int P_BYTES = 128 * 128;
constexpr int ATTN_SMEM = Q_BYTES + KV_STAGES * 2 * KV_TILE_BYTES + 2 * P_BYTES + 1024 + 256;
constexpr int ATTN_TMEM_COLS = 256;                // S0 S1 (64 fp32 columns each), O (64), 64 unused (allocations are powers of two)
constexpr float kRescaleBits = 8.f;

struct AttnParams {
  AttnPlan plan;
  const int* block_table;
  int max_blocks, n_blocks, Hq, Hkv, group, layer;
  bf16* out;            // [T, Hq*64]
  float* split_ws;      // partials of sliced items: [q-tile][kv head][slice][2 + 64][128 rows]
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

// ------------------------------------------------------------------------------------------------
// Plan: one CTA.  For every q-tile the KV tiles it can see and into how many slices that range is cut, then
// the flat list of (q-tile, slice) items with everything a CTA needs to run one.
__global__ void attn_plan_kernel(RowMeta rm, AttnPlan pl, int n_seqs, int tokens_per_tile, int target_items,
                                 int min_chunk, const int* tile_count, const int* status) {
  pdl_wait();
  pdl_launch_dependents();
  __shared__ int s_total;
  if (threadIdx.x == 0) s_total = 0;
  __syncthreads();
  if (*status) {
    if (threadIdx.x == 0) *pl.n_items = 0;
    return;
  }
  const int n_tiles = *tile_count;
  int my = 0;
  for (int s = threadIdx.x; s < n_seqs; s += blockDim.x) {
    const int t0 = rm.seq_tile0[s], t1 = rm.seq_tile0[s + 1];
    const int L = rm.seq_len[s], n = rm.seq_n[s];
    for (int t = t0; t < t1; ++t) {
      const int tok_end = min(n, (t - t0 + 1) * tokens_per_tile);
      const int n_kv = (L + tok_end + 63) >> 6;
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
      const int ns = max(1, min(kAttnMaxSplits, (n_kv + chunk - 1) / chunk));
      const int base = n_kv / ns, rem = n_kv % ns;
      int lo = 0;
      for (int k = 0; k < ns; ++k) {
        const int len = base + (k < rem ? 1 : 0);
        pl.items_unsorted[2 * n] = make_int4(rm.seq_q0[s] + tok0, rm.seq_len[s] + tok0,
                                             min(tokens_per_tile, rm.seq_n[s] - tok0), rm.seq_slot[s]);
        pl.items_unsorted[2 * n + 1] = make_int4(lo | ((lo + len) << 16), k | (ns << 8) | (tok0 << 16), t, len);
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
}

void launch_attn_plan(cudaStream_t st, const RowMeta& rm, const AttnPlan& pl, int n_seqs, int tokens_per_tile,
                      int target_items, int min_chunk, const int* tile_count, const int* status, bool pdl) {
  launch_kernel(attn_plan_kernel, dim3(1), dim3(256), 0, st, pdl, rm, pl, n_seqs, tokens_per_tile, target_items, min_chunk,
                tile_count, status);
}

// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kAttnThreads, 2)
attn_sm100_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                  const __grid_constant__ CUtensorMap tmV, AttnParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sQ = smem;
  uint8_t* sKV = sQ + Q_BYTES;                         // stage s: K at s*2*KV_TILE_BYTES, V right after
  uint8_t* sP = sKV + KV_STAGES * 2 * KV_TILE_BYTES;   // two P buffers
  uint64_t* bars = reinterpret_cast<uint64_t*>(sP + 2 * P_BYTES);
  uint64_t* q_full = bars;                 // Q tile landed                       (one phase per item)
  uint64_t* q_empty = bars + 1;            // every S MMA of the item has read Q   (one phase per item)
  uint64_t* kv_full = bars + 2;
  uint64_t* kv_empty = kv_full + KV_STAGES;
  uint64_t* s_full = kv_empty + KV_STAGES;
  uint64_t* s_empty = s_full + 2;
  uint64_t* p_full = s_empty + 2;
  uint64_t* pv_full = p_full + 2;          // [g & 1] O += P(g) V(g) has completed
  uint64_t* group_bar = pv_full + 2;       // the four softmax warps (slice hand-over)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(group_bar + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  volatile int* s_flag = abort_flag + 1;   // combine: "this CTA ran the last slice to finish"

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    mbar_init(q_full, 1);
    mbar_init(q_empty, 1);
    for (int s = 0; s < KV_STAGES; ++s) {
      mbar_init(kv_full + s, 1);
      mbar_init(kv_empty + s, 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(s_full + b, 1);
      mbar_init(s_empty + b, 4);
      mbar_init(p_full + b, 128);
      mbar_init(pv_full + b, 1);
    }
    mbar_init(group_bar, 4);
    *abort_flag = 0;
    fence_mbar_init();
    tma_prefetch_desc(&tmQ);
    tma_prefetch_desc(&tmK);
    tma_prefetch_desc(&tmV);
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, ATTN_TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  pdl_wait();               // q, the K/V rows of this step, the row metadata and the plan come from earlier kernels
  pdl_launch_dependents();

  const int total = (*p.status) ? 0 : *p.plan.n_items * p.Hkv;
  // Round r of the walk: CTA i takes item r G + i in even rounds and r G + (G - 1 - i) in odd ones (the list is
  // sorted longest first, so the CTA that drew a long item in one round draws a short one in the next).
  const int n_rounds = (total + (int)gridDim.x - 1) / (int)gridDim.x;
  // A launch with fewer items than CTAs leaves some SMs with one busy CTA (the grid is two CTAs per SM, and CTA b
  // shares its SM with CTA b + G/2 under the usual placement); a CTA that has its SM alone walks its tiles faster,
  // so the longest items go to those SMs and the others pair a long item with a short one.
  const int half_grid = (int)gridDim.x / 2;
  auto item_of_round = [&](int r) -> int {
    if (n_rounds == 1 && total > half_grid) {
      const int n_second = total - half_grid;          // busy CTAs in the second half of the grid
      const int bx = (int)blockIdx.x;
      if (bx < half_grid) return bx >= n_second ? bx - n_second : (half_grid - n_second) + bx;
      return bx - half_grid < n_second ? total - 1 - (bx - half_grid) : -1;
    }
    const int i = (r & 1) ? (int)gridDim.x - 1 - (int)blockIdx.x : (int)blockIdx.x;
    const int w = r * (int)gridDim.x + i;
    return w < total ? w : -1;
  };

  // Global tile counter g (all items of this CTA): S / P / PV buffer = g & 1, KV stage = g % KV_STAGES, and every
  // barrier's parity follows from how often g has used it; n counts items (Q hand-over barriers).
  if (warp == 0) {
    if (lane == 0) {
      uint32_t g = 0;
      int n = 0;
      for (int r = 0; r < n_rounds; ++r) {
        const int w = item_of_round(r);
        if (w < 0) continue;
        const int4 ia = p.plan.items[2 * (w / p.Hkv)], ib = p.plan.items[2 * (w / p.Hkv) + 1];
        const int kvh = w % p.Hkv;
        const int kt_lo = ib.x & 0xffff, kt_hi = ib.x >> 16;
        const int* bt = p.block_table + (size_t)ia.w * p.max_blocks;
        int phys = bt[kt_lo];
        if (!mbar_wait(q_empty, (n & 1) ^ 1u, abort_flag, p.status, 400)) goto done;
        mbar_expect_tx(q_full, Q_BYTES);
        tma_load_3d(sQ, &tmQ, q_full, 0, kvh * p.group, ia.x);
        for (int j = kt_lo; j < kt_hi; ++j, ++g) {
          const int phys_next = (j + 1 < kt_hi) ? bt[j + 1] : 0;      // block-table entry of the next tile, ahead of need
          const int st = g % KV_STAGES;
          if (!mbar_wait(kv_empty + st, ((g / KV_STAGES) & 1) ^ 1u, abort_flag, p.status, 401)) goto done;
          const int row = (((p.layer * p.n_blocks) + phys) * p.Hkv + kvh) * 64;
          uint8_t* k_dst = sKV + st * 2 * KV_TILE_BYTES;
          mbar_expect_tx(kv_full + st, 2 * KV_TILE_BYTES);
          tma_load_2d(k_dst, &tmK, kv_full + st, 0, row);
          tma_load_2d(k_dst + KV_TILE_BYTES, &tmV, kv_full + st, 0, row);
          phys = phys_next;
        }
        ++n;
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc = umma_idesc_bf16(64);
      constexpr uint32_t idesc_pv = umma_idesc_bf16(64, true);
      const uint32_t q_addr = smem_u32(sQ);
      uint32_t g = 0;
      int n = 0;
      for (int r = 0; r < n_rounds; ++r) {
        const int w = item_of_round(r);
        if (w < 0) continue;
        const int4 ib = p.plan.items[2 * (w / p.Hkv) + 1];
        const int n_it = (ib.x >> 16) - (ib.x & 0xffff);
        auto issue_s = [&](uint32_t gi) -> bool {
          const int st = gi % KV_STAGES;
          if (!mbar_wait(kv_full + st, (gi / KV_STAGES) & 1, abort_flag, p.status, 410)) return false;
          if (!mbar_wait(s_empty + (gi & 1), ((gi >> 1) & 1) ^ 1u, abort_flag, p.status, 411)) return false;
          tc_fence_after();
          const uint32_t k_addr = smem_u32(sKV + st * 2 * KV_TILE_BYTES);
          const uint32_t d = tmem_base + (gi & 1) * 64;
#pragma unroll
          for (int k = 0; k < 4; ++k)
            umma_bf16(d, umma_desc_sw128(q_addr + k * 32), umma_desc_sw128(k_addr + k * 32), idesc, k != 0);
          umma_commit(s_full + (gi & 1));
          return true;
        };
        if (!mbar_wait(q_full, n & 1, abort_flag, p.status, 412)) goto done;
        if (!issue_s(g)) goto done;
        if (n_it == 1) umma_commit(q_empty);
        for (int j = 0; j < n_it; ++j, ++g) {
          if (j + 1 < n_it) {
            if (!issue_s(g + 1)) goto done;
            if (j + 2 == n_it) umma_commit(q_empty);      // last S MMA of the item issued: Q is free once it completes
          }
          // P(g) is written, and whatever had to be done to the accumulator before this product is done
          if (!mbar_wait(p_full + (g & 1), (g >> 1) & 1, abort_flag, p.status, 413)) goto done;
          tc_fence_after();
          const int st = g % KV_STAGES;
          const uint32_t p_addr = smem_u32(sP + (g & 1) * P_BYTES);
          const uint32_t v_addr = smem_u32(sKV + st * 2 * KV_TILE_BYTES + KV_TILE_BYTES);
          const uint32_t d = tmem_base + 128;      // the item's accumulator: the first product of an item overwrites it
#pragma unroll
          for (int k = 0; k < 4; ++k)   // V [key][dim] is MN-major: a K step of 16 keys is 16 rows of 128 bytes
            umma_bf16(d, umma_desc_sw128(p_addr + k * 32), umma_desc_sw128(v_addr + k * 2048), idesc_pv,
                      (j != 0 || k != 0) ? 1u : 0u);
          umma_commit(kv_empty + st);
          umma_commit(pv_full + (g & 1));
        }
        ++n;
      }
      // every stage-release arrival must land before the CTA's shared memory can be handed on
      if (g > 0 && !mbar_wait(pv_full + ((g - 1) & 1), ((g - 1) >> 1) & 1, abort_flag, p.status, 414)) goto done;
    }
  } else {
    const int quarter = warp & 3;
    const int row = quarter * 32 + lane;               // q row of the tile = TMEM lane
    const int tok = row / p.group;
    const uint32_t t_lane = tmem_base + (uint32_t(quarter * 32) << 16);
    const float sc = 0.125f * 1.4426950408889634f;     // 1/sqrt(64) * log2(e)
    uint32_t g = 0, group_ph = 0;
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
      float m_ref = -INFINITY, l = 0.f;                  // exponent reference (log2 units, scaled) and row sum under it
      const uint32_t t_o = t_lane + 128;                 // this warp's lanes of the accumulator

      for (int j = kt_lo; j < kt_hi; ++j, ++g) {
        const int b = g & 1;
        bool ok = mbar_wait(s_full + b, (g >> 1) & 1, abort_flag, p.status, 420);
        if (!__all_sync(0xffffffffu, ok)) goto done;
        tc_fence_after();
        if (!warp_ok) {
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(s_empty + b);
          mbar_arrive(p_full + b);
          continue;
        }
        uint32_t s0[32], s1[32];
        tmem_ld32(t_lane + b * 64, s0);
        tmem_ld32(t_lane + b * 64 + 32, s1);
        tmem_ld_wait();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(s_empty + b);

        const int kbase = j * 64;
        if (p.anc) {
          if (kbase + 63 >= len0) {                       // the tile holds rows of this call
            // 32 bits of the row's visibility string from key position `pos` on: ones below the committed length,
            // the ancestry mask over the call's rows, zeros beyond them
            auto word = [&](int i) -> uint32_t {
              return i < 0 ? 0xffffffffu : i == 0 ? am.x : i == 1 ? am.y : i == 2 ? am.z : i == 3 ? am.w : 0u;
            };
            auto vis32 = [&](int pos) -> uint32_t {
              if (pos <= -32) return 0xffffffffu;
              if (pos >= 128) return 0u;
              const int wi = pos >> 5;                    // floor, also for negative positions
              return __funnelshift_r(word(wi), word(wi + 1), pos & 31);
            };
            const uint32_t v0 = vis32(kbase - len0), v1 = vis32(kbase - len0 + 32);
#pragma unroll
            for (int e = 0; e < 32; ++e) {
              if (!((v0 >> e) & 1u)) s0[e] = 0xff800000u;          // -inf
              if (!((v1 >> e) & 1u)) s1[e] = 0xff800000u;
            }
          }
        } else if (kbase + 63 > pos0) {                   // some row of the tile masks part of this KV tile
#pragma unroll
          for (int e = 0; e < 32; ++e) {
            if (kbase + e > pos_row) s0[e] = 0xff800000u;          // -inf
            if (kbase + 32 + e > pos_row) s1[e] = 0xff800000u;
          }
        }
        float mx = -INFINITY;
#pragma unroll
        for (int e = 0; e < 32; ++e) mx = max3(mx, __uint_as_float(s0[e]), __uint_as_float(s1[e]));
        mx *= sc;
        // The reference moves only when the maximum has outgrown it by more than kRescaleBits (or nothing has been
        // accumulated under it yet: then moving it costs nothing).
        float alpha = 1.f;
        bool rescale = false;
        if (mx > m_ref) {
          if (l == 0.f) {
            m_ref = mx;                                   // nothing accumulated so far (first tile, or all keys masked)
          } else if (mx > m_ref + kRescaleBits) {
            alpha = ex2(m_ref - mx);
            m_ref = mx;
            rescale = true;
          }
        }
        const float m_use = (m_ref == -INFINITY) ? 0.f : m_ref;
        float sum = 0.f;
        uint32_t pk[32];
#pragma unroll
        for (int e = 0; e < 16; ++e) {
          const float a0 = ex2(fmaf(__uint_as_float(s0[2 * e]), sc, -m_use));
          const float a1 = ex2(fmaf(__uint_as_float(s0[2 * e + 1]), sc, -m_use));
          sum += a0 + a1;
          pk[e] = pack_bf16(a0, a1);
        }
#pragma unroll
        for (int e = 0; e < 16; ++e) {
          const float a0 = ex2(fmaf(__uint_as_float(s1[2 * e]), sc, -m_use));
          const float a1 = ex2(fmaf(__uint_as_float(s1[2 * e + 1]), sc, -m_use));
          sum += a0 + a1;
          pk[16 + e] = pack_bf16(a0, a1);
        }
        l = l * alpha + sum;
        // P's buffer was last read by the product of tile g - 2: the only wait of the steady state, two tiles back
        if (g >= 2) {
          ok = mbar_wait(pv_full + b, ((g - 2) >> 1) & 1, abort_flag, p.status, 421);
          if (!__all_sync(0xffffffffu, ok)) goto done;
        }
        if (__any_sync(0xffffffffu, rescale)) {
          // rare: scale this warp's accumulator rows (alpha = 1 where not needed) once the product before this tile,
          // which still adds into them, has completed
          ok = mbar_wait(pv_full + (b ^ 1), ((g - 1) >> 1) & 1, abort_flag, p.status, 423);
          if (!__all_sync(0xffffffffu, ok)) goto done;
          tc_fence_after();
#pragma unroll
          for (int hf = 0; hf < 2; ++hf) {
            uint32_t o[32];
            tmem_ld32(t_o + hf * 32, o);
            tmem_ld_wait();
#pragma unroll
            for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
            tmem_st32(t_o + hf * 32, o);
          }
          tmem_st_wait();
          tc_fence_before();
        }
        // P row -> shared memory, K-major 128B-swizzled: 16-byte chunk c of row r sits at chunk c ^ (r & 7)
        uint8_t* prow = sP + b * P_BYTES + row * 128;
#pragma unroll
        for (int c = 0; c < 8; ++c)
          *reinterpret_cast<uint4*>(prow + ((c ^ (row & 7)) << 4)) =
              make_uint4(pk[4 * c], pk[4 * c + 1], pk[4 * c + 2], pk[4 * c + 3]);
        fence_proxy_async_smem();
        mbar_arrive(p_full + b);
      }
      // the item's last product (products complete in issue order, so all of them)
      if (warp_ok && kt_hi > kt_lo) {
        bool ok = mbar_wait(pv_full + ((g - 1) & 1), ((g - 1) >> 1) & 1, abort_flag, p.status, 422);
        if (!__all_sync(0xffffffffu, ok)) goto done;
        tc_fence_after();
      }

      // ---- item epilogue
      const int head = kvh * p.group + row % p.group;
      if (n_split == 1) {
        if (warp_ok) {                                     // (a whole warp reads tensor memory together)
          const float inv = 1.f / l;
          uint4* dst = reinterpret_cast<uint4*>(p.out + (size_t)(q_row0 + tok) * p.Hq * 64 + head * 64);
#pragma unroll
          for (int hf = 0; hf < 2; ++hf) {
            uint32_t o[32];
            tmem_ld32(t_o + hf * 32, o);
            tmem_ld_wait();
            if (row_ok) {
#pragma unroll
              for (int c = 0; c < 4; ++c)
                dst[hf * 4 + c] = make_uint4(
                    pack_bf16(__uint_as_float(o[8 * c]) * inv, __uint_as_float(o[8 * c + 1]) * inv),
                    pack_bf16(__uint_as_float(o[8 * c + 2]) * inv, __uint_as_float(o[8 * c + 3]) * inv),
                    pack_bf16(__uint_as_float(o[8 * c + 4]) * inv, __uint_as_float(o[8 * c + 5]) * inv),
                    pack_bf16(__uint_as_float(o[8 * c + 6]) * inv, __uint_as_float(o[8 * c + 7]) * inv));
            }
          }
          tc_fence_before();
        }
      } else {
        // partials of this (q-tile, kv head): [slice][66][128 rows] floats, entry 0 the exponent reference (log2
        // units), 1 the row sum under it, 2.. the 64 unnormalised outputs; a warp's accesses are 128-byte lines
        float* tile_part = p.split_ws + ((size_t)(ib.z * p.Hkv + kvh) * kAttnMaxSplits) * (66 * 128) + row;
        if (warp_ok) {
          float* part = tile_part + (size_t)split * (66 * 128);
          part[0] = m_ref;
          part[128] = l;
#pragma unroll
          for (int hf = 0; hf < 2; ++hf) {
            uint32_t o[32];
            tmem_ld32(t_o + hf * 32, o);
            tmem_ld_wait();
#pragma unroll
            for (int e = 0; e < 32; ++e) part[(2 + hf * 32 + e) * 128] = __uint_as_float(o[e]);
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
          for (int s = 0; s < n_split; ++s) M = fmaxf(M, __ldcg(tile_part + (size_t)s * (66 * 128)));
          float Lsum = 0.f;
          float o[64];
#pragma unroll
          for (int e = 0; e < 64; ++e) o[e] = 0.f;
          for (int s = 0; s < n_split; ++s) {             // fixed slice order: the result does not depend on arrival
            const float* ps = tile_part + (size_t)s * (66 * 128);
            const float mx = __ldcg(ps);
            const float wgt = (mx == -INFINITY) ? 0.f : ex2(mx - M);
            Lsum += wgt * __ldcg(ps + 128);
#pragma unroll
            for (int e = 0; e < 64; ++e) o[e] += wgt * __ldcg(ps + (2 + e) * 128);
          }
          if (row_ok) {
            const float inv = 1.f / Lsum;
            uint4* dst = reinterpret_cast<uint4*>(p.out + (size_t)(q_row0 + tok) * p.Hq * 64 + head * 64);
#pragma unroll
            for (int c = 0; c < 8; ++c)
              dst[c] = make_uint4(pack_bf16(o[8 * c] * inv, o[8 * c + 1] * inv), pack_bf16(o[8 * c + 2] * inv, o[8 * c + 3] * inv),
                                  pack_bf16(o[8 * c + 4] * inv, o[8 * c + 5] * inv), pack_bf16(o[8 * c + 6] * inv, o[8 * c + 7] * inv));
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
    tmem_dealloc(tmem_base, ATTN_TMEM_COLS);
  }
}

int launch_attn_sm100(cudaStream_t st, const CUtensorMap& tmQ, const CUtensorMap& tmK, const CUtensorMap& tmV,
                      const AttnPlan& plan, const KvView& kv, const ModelDims& md, int layer, bf16* out, int n_sms,
                      int device, int* status, float* split_ws, const uint4* anc, bool pdl) {
  static bool attr_set[kMaxDevices] = {};          // the attribute is per device
  if (device < 0 || device >= kMaxDevices) return -1;
  if (!attr_set[device]) {
    if (cudaFuncSetAttribute(attn_sm100_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, ATTN_SMEM) != cudaSuccess)
      return -1;
    attr_set[device] = true;
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
  return launch_kernel(attn_sm100_kernel, dim3(2 * n_sms), dim3(kAttnThreads), ATTN_SMEM, st, pdl, tmQ, tmK, tmV, p);
}

}  // namespace hsd
