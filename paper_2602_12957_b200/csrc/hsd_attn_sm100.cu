// Varlen multi-query-token causal attention over the paged KV cache, tcgen05 / TMEM / TMA (sm_100a).
//
// A draft token attends to every committed row of its sequence and, causally, to the draft rows before it
// (the chain case of the paper's tree-ancestry mask, Sec. 3.2 / Fig. 2(c)).
//
// Work item = (q-tile, kv head, kv split).  A q-tile is 128 MMA rows: 128/group consecutive tokens of one
// sequence x the `group` query heads that share the kv head (GQA packing, so K/V tiles are read once per
// group).  K tiles [64 keys][64 dims] and V^T tiles [64 dims][64 keys] are exactly one paged block per kv
// head, fetched by TMA through the block table.
//
// Warp roles: warp 0 = TMA producer, warp 1 = MMA issuer + TMEM owner, warps 2..5 = softmax (one TMEM lane
// quarter each, one thread per q row, no shuffles).  Per KV tile: S = Q K^T (TMEM) -> online softmax in
// registers -> P (bf16, shared memory, 128B-swizzled) -> PV = P V (TMEM) -> accumulated into registers with
// the running-max rescale.  S and PV are double-buffered so the tensor pipe works on tile j+1 while the
// softmax warps are on tile j; two CTAs per SM interleave further.
#include "hsd_kernels.h"

namespace hsd {

constexpr int kAttnThreads = 192;
constexpr int KV_STAGES = 3;
constexpr int Q_BYTES = 128 * 128;
constexpr int KV_TILE_BYTES = 64 * 128;            // one K tile or one V^T tile
constexpr int P_BYTES = 128 * 128;
constexpr int ATTN_SMEM = Q_BYTES + KV_STAGES * 2 * KV_TILE_BYTES + 2 * P_BYTES + 1024 + 256;
constexpr int ATTN_TMEM_COLS = 256;                // S0 S1 PV0 PV1, 64 fp32 columns each

struct AttnWork {       // one work item
  int seq, tok0, n_tok, kvh, kt_lo, kt_hi, split, n_split;
};

struct AttnParams {
  RowMeta rm;
  const int* block_table;
  int max_blocks, n_blocks, Hq, Hkv, group, layer;
  bf16* out;            // [T, Hq*64]
  float* split_ws;      // partial results when n_split > 1
  const int* tile_count;
  int* status;
  int n_seqs;
};

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__global__ void __launch_bounds__(kAttnThreads, 2)
attn_sm100_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                  const __grid_constant__ CUtensorMap tmV, AttnParams p) {
  pdl_wait();               // q, the K/V rows of this step and the row metadata come from earlier kernels
  pdl_launch_dependents();
  if (*p.status) return;
  const int tile_idx = blockIdx.x / p.Hkv;
  const int kvh = blockIdx.x % p.Hkv;
  if (tile_idx >= *p.tile_count) return;

  // locate the sequence of this q-tile: largest s with seq_tile0[s] <= tile_idx
  int lo = 0, hi = p.n_seqs - 1;
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (p.rm.seq_tile0[mid] <= tile_idx) lo = mid; else hi = mid - 1;
  }
  const int seq = lo;
  const int TOK = 128 / p.group;
  const int tok0 = (tile_idx - p.rm.seq_tile0[seq]) * TOK;
  const int n_tok = min(TOK, p.rm.seq_n[seq] - tok0);
  const int q_row0 = p.rm.seq_q0[seq] + tok0;
  const int pos0 = p.rm.seq_len[seq] + tok0;          // position of the tile's first token
  const int n_kv = (pos0 + n_tok + 63) >> 6;          // KV tiles this q-tile can see
  const int slot = p.rm.seq_slot[seq];

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sQ = smem;
  uint8_t* sKV = sQ + Q_BYTES;                         // stage s: K at s*2*KV_TILE_BYTES, V^T right after
  uint8_t* sP = sKV + KV_STAGES * 2 * KV_TILE_BYTES;   // two P buffers
  uint64_t* bars = reinterpret_cast<uint64_t*>(sP + 2 * P_BYTES);
  uint64_t* q_full = bars;
  uint64_t* kv_full = bars + 1;
  uint64_t* kv_empty = kv_full + KV_STAGES;
  uint64_t* s_full = kv_empty + KV_STAGES;
  uint64_t* s_empty = s_full + 2;
  uint64_t* p_full = s_empty + 2;
  uint64_t* pv_full = p_full + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(pv_full + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    mbar_init(q_full, 1);
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

  if (warp == 0) {
    if (lane == 0) {
      mbar_expect_tx(q_full, Q_BYTES);
      tma_load_3d(sQ, &tmQ, q_full, 0, kvh * p.group, q_row0);
      const int* bt = p.block_table + (size_t)slot * p.max_blocks;
      for (int j = 0; j < n_kv; ++j) {
        const int st = j % KV_STAGES;
        if (!mbar_wait(kv_empty + st, ((j / KV_STAGES) & 1) ^ 1u, abort_flag, p.status, 400)) goto done;
        const int phys = bt[j];
        const int row = (((p.layer * p.n_blocks) + phys) * p.Hkv + kvh) * 64;
        uint8_t* k_dst = sKV + st * 2 * KV_TILE_BYTES;
        mbar_expect_tx(kv_full + st, 2 * KV_TILE_BYTES);
        tma_load_2d(k_dst, &tmK, kv_full + st, 0, row);
        tma_load_2d(k_dst + KV_TILE_BYTES, &tmV, kv_full + st, 0, row);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc = umma_idesc_bf16(64);
      const uint32_t q_addr = smem_u32(sQ);
      auto issue_s = [&](int j) -> bool {
        const int st = j % KV_STAGES;
        if (!mbar_wait(kv_full + st, (j / KV_STAGES) & 1, abort_flag, p.status, 410)) return false;
        if (!mbar_wait(s_empty + (j & 1), ((j >> 1) & 1) ^ 1u, abort_flag, p.status, 411)) return false;
        tc_fence_after();
        const uint32_t k_addr = smem_u32(sKV + st * 2 * KV_TILE_BYTES);
        const uint32_t d = tmem_base + (j & 1) * 64;
#pragma unroll
        for (int k = 0; k < 4; ++k)
          umma_bf16(d, umma_desc_sw128(q_addr + k * 32), umma_desc_sw128(k_addr + k * 32), idesc, k != 0);
        umma_commit(s_full + (j & 1));
        return true;
      };
      if (!mbar_wait(q_full, 0, abort_flag, p.status, 412)) goto done;
      if (!issue_s(0)) goto done;
      for (int j = 0; j < n_kv; ++j) {
        if (j + 1 < n_kv && !issue_s(j + 1)) goto done;
        if (!mbar_wait(p_full + (j & 1), (j >> 1) & 1, abort_flag, p.status, 413)) goto done;
        tc_fence_after();
        const int st = j % KV_STAGES;
        const uint32_t p_addr = smem_u32(sP + (j & 1) * P_BYTES);
        const uint32_t v_addr = smem_u32(sKV + st * 2 * KV_TILE_BYTES + KV_TILE_BYTES);
        const uint32_t d = tmem_base + 128 + (j & 1) * 64;
#pragma unroll
        for (int k = 0; k < 4; ++k)
          umma_bf16(d, umma_desc_sw128(p_addr + k * 32), umma_desc_sw128(v_addr + k * 32), idesc, k != 0);
        umma_commit(kv_empty + st);
        umma_commit(pv_full + (j & 1));
      }
      // the last stage-release arrival must land before the CTA's shared memory can be handed on
      if (!mbar_wait(kv_empty + (n_kv - 1) % KV_STAGES, ((n_kv - 1) / KV_STAGES) & 1, abort_flag, p.status, 414))
        goto done;
    }
  } else {
    const int quarter = warp & 3;
    const int row = quarter * 32 + lane;               // q row of the tile = TMEM lane
    const int tok = row / p.group;
    const int pos_row = pos0 + tok;
    const bool row_ok = tok < n_tok;
    const uint32_t t_lane = tmem_base + (uint32_t(quarter * 32) << 16);
    const float sc = 0.125f * 1.4426950408889634f;     // 1/sqrt(64) * log2(e)
    float m = -INFINITY, l = 0.f, alpha_prev = 1.f;
    float o[64];
#pragma unroll
    for (int e = 0; e < 64; ++e) o[e] = 0.f;

    for (int j = 0; j <= n_kv; ++j) {
      if (j < n_kv) {
        const int b = j & 1;
        bool ok = mbar_wait(s_full + b, (j >> 1) & 1, abort_flag, p.status, 420);
        if (!__all_sync(0xffffffffu, ok)) goto done;
        tc_fence_after();
        uint32_t s0[32], s1[32];
        tmem_ld32(t_lane + b * 64, s0);
        tmem_ld32(t_lane + b * 64 + 32, s1);
        tmem_ld_wait();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(s_empty + b);

        const int kbase = j * 64;
        const bool diag = kbase + 63 > pos0;             // some row of the tile masks part of this KV tile
        float mx = -INFINITY;
        if (diag) {
#pragma unroll
          for (int e = 0; e < 32; ++e) {
            if (kbase + e > pos_row) s0[e] = 0xff800000u;          // -inf
            if (kbase + 32 + e > pos_row) s1[e] = 0xff800000u;
          }
        }
#pragma unroll
        for (int e = 0; e < 32; ++e) mx = fmaxf(mx, fmaxf(__uint_as_float(s0[e]), __uint_as_float(s1[e])));
        const float m_new = fmaxf(m, mx * sc);
        const float m_use = (m_new == -INFINITY) ? 0.f : m_new;
        const float alpha = ex2(m - m_use);
        float sum = 0.f;
        uint32_t pk[32];
#pragma unroll
        for (int e = 0; e < 16; ++e) {
          const float a0 = ex2(__uint_as_float(s0[2 * e]) * sc - m_use);
          const float a1 = ex2(__uint_as_float(s0[2 * e + 1]) * sc - m_use);
          sum += a0 + a1;
          pk[e] = pack_bf16(a0, a1);
        }
#pragma unroll
        for (int e = 0; e < 16; ++e) {
          const float a0 = ex2(__uint_as_float(s1[2 * e]) * sc - m_use);
          const float a1 = ex2(__uint_as_float(s1[2 * e + 1]) * sc - m_use);
          sum += a0 + a1;
          pk[16 + e] = pack_bf16(a0, a1);
        }
        l = l * alpha + sum;
        // P row -> shared memory, K-major 128B-swizzled: 16-byte chunk c of row r sits at chunk c ^ (r & 7)
        uint8_t* prow = sP + b * P_BYTES + row * 128;
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          uint4 v = make_uint4(pk[4 * c], pk[4 * c + 1], pk[4 * c + 2], pk[4 * c + 3]);
          *reinterpret_cast<uint4*>(prow + ((c ^ (row & 7)) << 4)) = v;
        }
        fence_proxy_async_smem();
        mbar_arrive(p_full + b);
        m = m_new;
        // the rescale for everything accumulated so far is applied when PV(j-1) is folded in below
        if (j > 0) {
          const int pb = (j - 1) & 1;
          ok = mbar_wait(pv_full + pb, ((j - 1) >> 1) & 1, abort_flag, p.status, 421);
          if (!__all_sync(0xffffffffu, ok)) goto done;
          tc_fence_after();
          uint32_t t0[32], t1[32];
          tmem_ld32(t_lane + 128 + pb * 64, t0);
          tmem_ld32(t_lane + 128 + pb * 64 + 32, t1);
          tmem_ld_wait();
#pragma unroll
          for (int e = 0; e < 32; ++e) {
            o[e] = o[e] * alpha_prev + __uint_as_float(t0[e]);
            o[32 + e] = o[32 + e] * alpha_prev + __uint_as_float(t1[e]);
          }
        }
        alpha_prev = alpha;
      } else {
        const int pb = (j - 1) & 1;
        bool ok = mbar_wait(pv_full + pb, ((j - 1) >> 1) & 1, abort_flag, p.status, 422);
        if (!__all_sync(0xffffffffu, ok)) goto done;
        tc_fence_after();
        uint32_t t0[32], t1[32];
        tmem_ld32(t_lane + 128 + pb * 64, t0);
        tmem_ld32(t_lane + 128 + pb * 64 + 32, t1);
        tmem_ld_wait();
#pragma unroll
        for (int e = 0; e < 32; ++e) {
          o[e] = o[e] * alpha_prev + __uint_as_float(t0[e]);
          o[32 + e] = o[32 + e] * alpha_prev + __uint_as_float(t1[e]);
        }
      }
    }
    if (row_ok) {
      const float inv = 1.f / l;
      const int head = kvh * p.group + row % p.group;
      uint4* dst = reinterpret_cast<uint4*>(p.out + (size_t)(q_row0 + tok) * p.Hq * 64 + head * 64);
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        uint4 v;
        v.x = pack_bf16(o[8 * c + 0] * inv, o[8 * c + 1] * inv);
        v.y = pack_bf16(o[8 * c + 2] * inv, o[8 * c + 3] * inv);
        v.z = pack_bf16(o[8 * c + 4] * inv, o[8 * c + 5] * inv);
        v.w = pack_bf16(o[8 * c + 6] * inv, o[8 * c + 7] * inv);
        dst[c] = v;
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
                        const RowMeta& rm, const KvView& kv, const ModelDims& md, int layer, bf16* out, int n_seqs,
                        int max_tiles, const int* tile_count, int* status, float* split_ws, bool pdl) {
  static bool attr_set = false;
  if (!attr_set) {
    if (cudaFuncSetAttribute(attn_sm100_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, ATTN_SMEM) != cudaSuccess)
      return -1;
    attr_set = true;
  }
  AttnParams p;
  p.rm = rm;
  p.block_table = kv.block_table;
  p.max_blocks = kv.max_blocks;
  p.n_blocks = kv.n_blocks;
  p.Hq = md.Hq;
  p.Hkv = md.Hkv;
  p.group = md.group;
  p.layer = layer;
  p.out = out;
  p.split_ws = split_ws;
  p.tile_count = tile_count;
  p.status = status;
  p.n_seqs = n_seqs;
  return launch_kernel(attn_sm100_kernel, dim3(max_tiles * md.Hkv), dim3(kAttnThreads), ATTN_SMEM, st, pdl, tmQ, tmK, tmV,
                       p);
}

}  // namespace hsd
