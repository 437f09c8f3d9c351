// tcgen05 / TMEM GEMM for sm_100a:  C = A W^T,  A [M,K] bf16 (activations), W [n_out,K] bf16 (weights),
// fp32 accumulation in tensor memory, operands staged in shared memory by TMA (128-byte swizzle).
//
// One persistent CTA per SM walks work units (128 x BN output tile, optionally one slice of K), M fastest so
// CTAs running side by side share a weight tile through L2.  Warp roles:
//   warp 0      A producer (one lane): activation tile, one 128-row TMA box per stage
//   warp 1      MMA issuer (one lane) and TMEM owner
//   warps 2, 3  B producers (one lane each): the two halves of the weight tile, one TMA box each per stage.
//               A TMA instruction costs its issuing thread ~0.25 us whatever the box size, so a stage is three
//               large boxes issued from three warps instead of many small ones from one.  Weights do not depend
//               on the previous kernel, so these two start before the programmatic-launch wait.
//   warps 4..7  epilogue, one TMEM lane quarter each
// Two accumulator buffers in TMEM let the epilogue of unit i overlap the main loop of unit i+1.
//
// Epilogues (all fused; results leave the SM through swizzled staging buffers and TMA stores, so global
// writes are full 128-byte lines whatever the thread-to-row mapping in TMEM):
//   GS_STORE_BF16  C bf16 = acc
//   GS_ADD_F32     C fp32 += acc   (TMA reduce-add into the residual stream; with split-K every K slice adds)
//   GS_SWIGLU      C bf16 = silu(gate) * up              (gate rows and up rows of W land in one tile)
//   GS_ARGMAX      per-row running argmax over the vocabulary + the next draft token's logit; logits never
//                  leave the SM (Eq. 10 of the paper fused into the LM head)
//   GS_QKV_ROPE    rotary embedding on q and k heads, q -> packed bf16, k/v -> paged KV pool (head_dim 64;
//                  GS_QKV_ROPE128: the same for head_dim 128)
#include "hsd_kernels.h"

namespace hsd {

// ------------------------------------------------------------------------------------------------
// driver entry point for tensor-map encoding (resolved at run time; the library does not link libcuda)
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static EncodeTiledFn g_encode = nullptr;

int tma_init() {
  if (g_encode) return 0;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
  if (e != cudaSuccess || qres != cudaDriverEntryPointSuccess || !fn) return -1;
  g_encode = reinterpret_cast<EncodeTiledFn>(fn);
  return 0;
}

int make_tmap_2d(CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
  if (!g_encode) return -1;
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {cols * 2};
  cuuint32_t box[2] = {64, box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = g_encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? 0 : -1;
}

int make_tmap_2d_f32(CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
  if (!g_encode) return -1;
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {cols * 4};
  cuuint32_t box[2] = {32, box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = g_encode(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void*>(base), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? 0 : -1;
}

int make_tmap_3d(CUtensorMap* map, const void* base, uint64_t d0, uint64_t d1, uint64_t d2, uint64_t stride1_bytes,
                 uint64_t stride2_bytes, uint32_t b0, uint32_t b1, uint32_t b2) {
  if (!g_encode) return -1;
  cuuint64_t dims[3] = {d0, d1, d2};
  cuuint64_t strides[2] = {stride1_bytes, stride2_bytes};
  cuuint32_t box[3] = {b0, b1, b2};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = g_encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? 0 : -1;
}

int make_weight_tmaps(WeightMaps* w, const void* base, uint64_t rows, uint64_t cols) {
  int bad = 0;
  for (int i = 0; i < 3; ++i) bad |= make_tmap_2d(&w->m[i], base, rows, cols, 32u << i);
  return bad;
}

// ------------------------------------------------------------------------------------------------
// K extent of a pipeline stage in 64-column sub-tiles.  Two (one barrier round trip per eight MMAs instead of four)
// measured the same cycles per k-block as one: with 256-wide tiles the main loop runs at the tensor pipes' rate.
#ifndef HSD_GEMM_KSTEPS
#define HSD_GEMM_KSTEPS 1
#endif
constexpr int BM = 128;
constexpr int KSUB = 64;                         // one 128-byte-swizzled sub-tile spans 64 bf16 of K
constexpr int KSTEPS = HSD_GEMM_KSTEPS;          // sub-tiles per pipeline stage
constexpr int BK = KSUB * KSTEPS;                // K extent of one stage (one barrier round trip)
constexpr int A_SUB = BM * KSUB * 2;             // bytes of one A sub-tile
constexpr int A_BYTES = A_SUB * KSTEPS;
constexpr int kGemmThreads = 256;
constexpr int STG_BYTES = 4096;                  // one epilogue staging buffer: 32 rows x 128 bytes
constexpr int STG_TOTAL = 4 * 2 * STG_BYTES;     // four epilogue warps, two buffers each

// PAIR: two CTAs (a cluster) share one 256 x BN tile: each stages its own 128 rows of A and BN/2 rows of B.
#ifndef HSD_GEMM_STAGES_PAIR
#define HSD_GEMM_STAGES_PAIR (6 / KSTEPS)
#define HSD_GEMM_STAGES_256 (4 / KSTEPS)
#define HSD_GEMM_STAGES_128 (6 / KSTEPS)
#define HSD_GEMM_STAGES_64 (8 / KSTEPS)
#endif
template <int BN, bool PAIR = false>
struct Cfg {
  static constexpr int B_SUB = (PAIR ? BN / 2 : BN) * KSUB * 2;     // bytes of one B sub-tile this CTA stages
  static constexpr int B_BYTES = B_SUB * KSTEPS;                    // bytes of B per stage
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int STAGES = PAIR ? HSD_GEMM_STAGES_PAIR
                                     : ((BN == 256) ? HSD_GEMM_STAGES_256 : (BN == 128 ? HSD_GEMM_STAGES_128 : HSD_GEMM_STAGES_64));
  static constexpr int TMEM_COLS = 2 * BN;
  static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + STG_TOTAL + 1024 /*alignment slack*/ + 256 /*barriers*/;
};

struct GemmDev {
  int M, n_cols, K, n_up_off;   // n_cols: output columns; n_up_off: row offset of the `up` half (SwiGLU)
  int splits, kb_per_split;     // K slices per tile (GS_ADD_F32 only) and k-blocks per slice
  GemmOut out;
  QkvEpilogue qkv;
  int* status;
};

// TMA store / reduce of one staging buffer and the bulk-group bookkeeping around it (issued by one lane).
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, const void* smem_src, int x, int y) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
               ::"l"(reinterpret_cast<uint64_t>(map)), "r"(smem_u32(smem_src)), "r"(x), "r"(y)
               : "memory");
}
__device__ __forceinline__ void tma_reduce_add_2d(const CUtensorMap* map, const void* smem_src, int x, int y) {
  asm volatile("cp.reduce.async.bulk.tensor.2d.global.shared::cta.add.bulk_group [%0, {%2, %3}], [%1];"
               ::"l"(reinterpret_cast<uint64_t>(map)), "r"(smem_u32(smem_src)), "r"(x), "r"(y)
               : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_read() {
  asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}


// 16-byte chunk `c` of this lane's 128-byte staging row, at its 128-byte-swizzle position.
__device__ __forceinline__ uint4* stg_chunk(uint8_t* buf, int lane, int c) {
  return reinterpret_cast<uint4*>(buf + lane * 128 + ((c ^ (lane & 7)) << 4));
}
__device__ __forceinline__ uint4 pack8(const uint32_t* r) {
  uint4 o;
  o.x = pack_bf16(__uint_as_float(r[0]), __uint_as_float(r[1]));
  o.y = pack_bf16(__uint_as_float(r[2]), __uint_as_float(r[3]));
  o.z = pack_bf16(__uint_as_float(r[4]), __uint_as_float(r[5]));
  o.w = pack_bf16(__uint_as_float(r[6]), __uint_as_float(r[7]));
  return o;
}

template <int BN, int MODE, bool PAIR>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_sm100_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                  const __grid_constant__ CUtensorMap tmC, GemmDev p) {
  using C = Cfg<BN, PAIR>;
  constexpr int OUT_N = (MODE == GS_SWIGLU) ? BN / 2 : BN;   // output columns per tile
  constexpr int HALF_B = BN / 2 * KSUB * 2;                  // bytes of one weight half-tile of one sub-tile
  constexpr int TILE_M = PAIR ? 2 * BM : BM;                 // rows of one work unit (both CTAs of a pair)
  const int rank = PAIR ? (int)cluster_ctarank() : 0;        // 0 = the CTA that issues the MMAs
  const int cta = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;       // index among the unit walkers
  const int n_cta = PAIR ? (int)(gridDim.x >> 1) : (int)gridDim.x;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* stg = smem + C::STAGES * C::STAGE_BYTES;
  uint64_t* bars = reinterpret_cast<uint64_t*>(stg + STG_TOTAL);
  uint64_t* full = bars;
  uint64_t* empty = bars + C::STAGES;
  uint64_t* tfull = bars + 2 * C::STAGES;
  uint64_t* tempty = tfull + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tempty + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < C::STAGES; ++s) {
      // A producer + two B producers, each with its own byte count; a pair: one arrival (even CTA) for all bytes
      mbar_init(full + s, PAIR ? 1 : 3);
      mbar_init(empty + s, 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(tfull + b, 1);
      mbar_init(tempty + b, PAIR ? 8 : 4);     // the epilogue warps of both CTAs release the even CTA's MMA thread
    }
    *abort_flag = 0;
    fence_mbar_init();
    tma_prefetch_desc(&tmA);
    tma_prefetch_desc(&tmB);
    if (MODE != GS_ARGMAX) tma_prefetch_desc(&tmC);
  }
  if (warp == 1) {
    if (PAIR) {
      tmem_alloc_pair(tmem_slot, C::TMEM_COLS);
      tmem_relinquish_pair();
    } else {
      tmem_alloc(tmem_slot, C::TMEM_COLS);
      tmem_relinquish();
    }
  }
  tc_fence_before();
  __syncthreads();
  if (PAIR) cluster_sync();          // both CTAs' barriers exist before either one's loads complete on them
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  const int m_tiles = (p.M + TILE_M - 1) / TILE_M;
  const int n_tiles = p.n_cols / OUT_N;
  const int tiles = m_tiles * n_tiles;
  const int total = tiles * p.splits;
  const int k_blocks = p.K / BK;

  // Producer warps: lanes 0 and 1 each take every other stage (kc counts k-blocks over all units of this CTA;
  // the stage count is even, so a lane always sees the same stages).  One thread cannot issue TMA instructions
  // faster than about one per 0.25 us, and a barrier round trip adds to that; two lanes per operand keep the
  // issue interval below the 128 x 256 MMA time of a k-block.
  if (warp == 0) {
    // ---- A producer: activations, written by the previous kernel
    if (lane < 2) {
      pdl_wait();
      if (lane == 0) pdl_launch_dependents();
      int kc = 0;
      for (int t = cta; t < total; t += n_cta) {
        const int tile = t % tiles, split = t / tiles;
        const int m0 = (tile % m_tiles) * TILE_M + rank * BM;
        const int kb0 = split * p.kb_per_split, kb1 = min(k_blocks, kb0 + p.kb_per_split);
        for (int kb = kb0; kb < kb1; ++kb, ++kc) {
          if ((kc & 1) != lane) continue;
          const int s = kc % C::STAGES;
          const uint32_t ph = (kc / C::STAGES) & 1;
          if (!mbar_wait(empty + s, ph ^ 1u, abort_flag, p.status, 100)) goto done;
          if (PAIR) {
            if (rank == 0) mbar_expect_tx(full + s, 2 * C::STAGE_BYTES);   // A and B of both CTAs land on this barrier
#pragma unroll
            for (int u = 0; u < KSTEPS; ++u)
              tma_load_2d_pair(smem + s * C::STAGE_BYTES + u * A_SUB, &tmA, full + s, kb * BK + u * KSUB, m0);
          } else {
            mbar_expect_tx(full + s, A_BYTES);
#pragma unroll
            for (int u = 0; u < KSTEPS; ++u)
              tma_load_2d(smem + s * C::STAGE_BYTES + u * A_SUB, &tmA, full + s, kb * BK + u * KSUB, m0);
          }
        }
      }
    }
  } else if (warp == 2 || warp == 3) {
    // ---- B producers: one half of the weight tile each (for SwiGLU: gate rows / up rows)
    if (lane < 2 && !(PAIR && warp == 3)) {
      // a pair: this CTA stages half `rank` of the tile in one box; alone: warps 2 and 3 stage one half each
      const int half = PAIR ? rank : warp - 2;
      int kc = 0;
      for (int t = cta; t < total; t += n_cta) {
        const int tile = t % tiles, split = t / tiles;
        const int n0 = (tile / m_tiles) * OUT_N;
        const int kb0 = split * p.kb_per_split, kb1 = min(k_blocks, kb0 + p.kb_per_split);
        const int row = (MODE == GS_SWIGLU) ? (half ? p.n_up_off + n0 : n0) : n0 + half * (BN / 2);
        for (int kb = kb0; kb < kb1; ++kb, ++kc) {
          if ((kc & 1) != lane) continue;
          const int s = kc % C::STAGES;
          const uint32_t ph = (kc / C::STAGES) & 1;
          if (!mbar_wait(empty + s, ph ^ 1u, abort_flag, p.status, 110 + half)) goto done;
          if (PAIR) {
#pragma unroll
            for (int u = 0; u < KSTEPS; ++u)
              tma_load_2d_pair(smem + s * C::STAGE_BYTES + A_BYTES + u * C::B_SUB, &tmB, full + s, kb * BK + u * KSUB, row);
          } else {
            mbar_expect_tx(full + s, HALF_B * KSTEPS);
#pragma unroll
            for (int u = 0; u < KSTEPS; ++u)
              tma_load_2d(smem + s * C::STAGE_BYTES + A_BYTES + u * C::B_SUB + half * HALF_B, &tmB, full + s,
                          kb * BK + u * KSUB, row);
          }
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc = umma_idesc_bf16(BN, false, TILE_M);
      int s = 0;
      uint32_t ph = 0;
      int it = 0;
      for (int t = cta; t < total; t += n_cta, ++it) {
        const int split = t / tiles;
        const int kb0 = split * p.kb_per_split, kb1 = min(k_blocks, kb0 + p.kb_per_split);
        const int b = it & 1;
        const uint32_t aph = (it >> 1) & 1;
        if (!mbar_wait(tempty + b, aph ^ 1u, abort_flag, p.status, 200)) goto done;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + b * BN;
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!mbar_wait(full + s, ph, abort_flag, p.status, 201)) goto done;
          tc_fence_after();
          const uint32_t sa = smem_u32(smem + s * C::STAGE_BYTES);
          const uint32_t sb = sa + A_BYTES;
#pragma unroll
          for (int u = 0; u < KSTEPS; ++u) {
#pragma unroll
            for (int k = 0; k < KSUB / 16; ++k) {
              const uint32_t acc = (kb != kb0 || u != 0 || k != 0) ? 1u : 0u;
              const uint64_t da = umma_desc_sw128(sa + u * A_SUB + k * 32), db = umma_desc_sw128(sb + u * C::B_SUB + k * 32);
              if (PAIR) umma_bf16_pair(d_tmem, da, db, idesc, acc);
              else umma_bf16(d_tmem, da, db, idesc, acc);
            }
          }
          // smem stage reusable once these MMAs have read it (in both CTAs of a pair)
          if (PAIR) umma_commit_pair(empty + s); else umma_commit(empty + s);
          if (++s == C::STAGES) { s = 0; ph ^= 1u; }
        }
        if (PAIR) umma_commit_pair(tfull + b); else umma_commit(tfull + b);   // accumulator complete
      }
    }
  } else {
    // ---- epilogue warps 4..7
    const int quarter = warp & 3;                 // TMEM lanes [32*quarter, +32) belong to this warp
    const int row_in_tile = quarter * 32 + lane;
    uint8_t* my_stg = stg + quarter * 2 * STG_BYTES;
    int n_stores = 0;                             // staging buffers handed to TMA so far (selects the buffer)
    pdl_wait();
    int it = 0;
    for (int t = cta; t < total; t += n_cta, ++it) {
      const int b = it & 1;
      const uint32_t aph = (it >> 1) & 1;
      const int tile = t % tiles;
      const int m0 = (tile % m_tiles) * TILE_M + rank * BM, n0 = (tile / m_tiles) * OUT_N;
      const int row = m0 + row_in_tile;
      const bool row_ok = row < p.M;
      const int wrow0 = m0 + quarter * 32;        // first row of this warp's 32-row slab
      const bool slab_ok = wrow0 < p.M;           // warp-uniform: the slab has at least one real row
      // rotary (cos, sin) of this thread's row: fetched while the main loop still runs, reused by every head
      float4 cs[MODE == GS_QKV_ROPE ? 16 : 1];
      if (MODE == GS_QKV_ROPE && row_ok) {
        const float4* src = reinterpret_cast<const float4*>(p.qkv.rope_cs + (size_t)row * 32);
#pragma unroll
        for (int i = 0; i < 16; ++i) cs[i] = __ldg(src + i);
      }
      // likewise the two words the K/V stores depend on (read here, used after the accumulator is ready).  row_kv
      // comes from the step's set-up kernel: after a failed device-side check it was not written, so nothing is
      // stored through it (q included: the step is a no-op), nor through a row outside the pool
      bool live = true;
      int phys = 0;
      int nxt = -1;                                 // LM head: the row's next draft token (its logit is captured)
      if (MODE == GS_ARGMAX) nxt = (row_ok && p.out.row_next) ? p.out.row_next[row] : -1;
      if (MODE == GS_QKV_ROPE || MODE == GS_QKV_ROPE128) {
        const int st_word = p.status ? *p.status : 0;
        const int kv_row = row_ok ? p.qkv.row_kv[row] : 0;
        live = st_word == 0;
        phys = live ? kv_row : 0;
      }
      bool ok = mbar_wait(tfull + b, aph, abort_flag, p.status, 300);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) goto done;
      tc_fence_after();
      const uint32_t t_acc = tmem_base + (uint32_t(quarter * 32) << 16) + b * BN;

      // A slab wholly beyond M stages nothing: every staged chunk commits exactly one bulk group, which is what
      // lets "at most one group pending" protect the buffer about to be rewritten.
      if (MODE == GS_STORE_BF16) {
#pragma unroll 1
        for (int c = 0; slab_ok && c < BN; c += 64) {
          uint8_t* buf = my_stg + (n_stores & 1) * STG_BYTES;
          if (lane == 0) bulk_wait_read<1>();      // the store that last read this buffer has drained
          __syncwarp();
          uint32_t r0[32], r1[32];
          tmem_ld32(t_acc + c, r0);
          tmem_ld32(t_acc + c + 32, r1);
          tmem_ld_wait();
#pragma unroll
          for (int v = 0; v < 4; ++v) {
            *stg_chunk(buf, lane, v) = pack8(r0 + 8 * v);
            *stg_chunk(buf, lane, 4 + v) = pack8(r1 + 8 * v);
          }
          fence_proxy_async_smem();
          __syncwarp();
          if (lane == 0) {
            tma_store_2d(&tmC, buf, n0 + c, wrow0);
            bulk_commit();
          }
          ++n_stores;
        }
      } else if (MODE == GS_ADD_F32) {
#pragma unroll 1
        for (int c = 0; slab_ok && c < BN; c += 32) {
          uint8_t* buf = my_stg + (n_stores & 1) * STG_BYTES;
          if (lane == 0) bulk_wait_read<1>();
          __syncwarp();
          uint32_t r[32];
          tmem_ld32(t_acc + c, r);
          tmem_ld_wait();
#pragma unroll
          for (int v = 0; v < 8; ++v)
            *stg_chunk(buf, lane, v) = make_uint4(r[4 * v], r[4 * v + 1], r[4 * v + 2], r[4 * v + 3]);
          fence_proxy_async_smem();
          __syncwarp();
          if (lane == 0) {
            tma_reduce_add_2d(&tmC, buf, n0 + c, wrow0);
            bulk_commit();
          }
          ++n_stores;
        }
      } else if (MODE == GS_SWIGLU) {
#pragma unroll 1
        for (int c = 0; slab_ok && c < OUT_N; c += 64) {
          uint8_t* buf = my_stg + (n_stores & 1) * STG_BYTES;
          if (lane == 0) bulk_wait_read<1>();
          __syncwarp();
#pragma unroll
          for (int hf = 0; hf < 2; ++hf) {
            uint32_t g[32], u[32];
            tmem_ld32(t_acc + c + hf * 32, g);
            tmem_ld32(t_acc + OUT_N + c + hf * 32, u);
            tmem_ld_wait();
#pragma unroll
            for (int e = 0; e < 32; ++e) {
              // silu(g) * u; the approximate divide (reciprocal + multiply, 2 ulp) has no slow-path branch, so the
              // 32 elements interleave; the result is rounded to bf16 anyway
              const float gv = __uint_as_float(g[e]);
              g[e] = __float_as_uint(__fdividef(gv, 1.f + __expf(-gv)) * __uint_as_float(u[e]));
            }
#pragma unroll
            for (int v = 0; v < 4; ++v) *stg_chunk(buf, lane, hf * 4 + v) = pack8(g + 8 * v);
          }
          fence_proxy_async_smem();
          __syncwarp();
          if (lane == 0) {
            tma_store_2d(&tmC, buf, n0 + c, wrow0);
            bulk_commit();
          }
          ++n_stores;
        }
      } else if (MODE == GS_ARGMAX) {
        float best_v = -INFINITY, zd = 0.f;
        int best_c = n0;
#pragma unroll 1
        for (int c = 0; c < BN; c += 32) {
          uint32_t r[32];
          tmem_ld32(t_acc + c, r);
          tmem_ld_wait();
#pragma unroll
          for (int e = 0; e < 32; ++e) {
            const float v = __uint_as_float(r[e]);
            const int col = n0 + c + e;
            if (v > best_v) { best_v = v; best_c = col; }
            if (col == nxt) zd = v;
          }
        }
        if (row_ok) {
          atomicMax(p.out.row_best + row, argmax_key(best_v, best_c));
          if (nxt >= n0 && nxt < n0 + BN) p.out.zdraft[row] = zd;
        }
      } else if (MODE == GS_QKV_ROPE) {
        const bool kv_ok = live && phys >= 0 && phys < p.qkv.kv_rows;
        if (!kv_ok) phys = 0;
        const int blk = phys >> 6, off = phys & 63;
#pragma unroll 1
        for (int hh = 0; hh < BN / 64; ++hh) {
          const int head = n0 / 64 + hh;
          const bool is_q = head < p.qkv.Hq;
          if (!slab_ok) break;
          uint8_t* buf = my_stg + (n_stores & 1) * STG_BYTES;
          if (is_q) {
            if (lane == 0) bulk_wait_read<1>();
            __syncwarp();
          }
          uint32_t lo[32], hi[32];
          tmem_ld32(t_acc + hh * 64, lo);
          tmem_ld32(t_acc + hh * 64 + 32, hi);
          tmem_ld_wait();
          if (p.qkv.q_norm && head < p.qkv.Hq + p.qkv.Hkv && row_ok) {
            // per-head RMSNorm of q and k over the head's 64 dims (all in this thread) before the rotation
            float ss = 0.f;
#pragma unroll
            for (int i = 0; i < 32; ++i)
              ss += __uint_as_float(lo[i]) * __uint_as_float(lo[i]) + __uint_as_float(hi[i]) * __uint_as_float(hi[i]);
            const float rs = rsqrtf(ss * (1.f / 64.f) + p.qkv.eps);
            const uint4* g4 = reinterpret_cast<const uint4*>(is_q ? p.qkv.q_norm : p.qkv.k_norm);
#pragma unroll
            for (int v = 0; v < 4; ++v) {
              const uint4 gl = __ldg(g4 + v), gh = __ldg(g4 + 4 + v);
              const uint32_t wl[4] = {gl.x, gl.y, gl.z, gl.w}, wh[4] = {gh.x, gh.y, gh.z, gh.w};
#pragma unroll
              for (int k = 0; k < 4; ++k) {
                lo[8 * v + 2 * k] = __float_as_uint(__uint_as_float(lo[8 * v + 2 * k]) * rs * bf16_lo(wl[k]));
                lo[8 * v + 2 * k + 1] = __float_as_uint(__uint_as_float(lo[8 * v + 2 * k + 1]) * rs * bf16_hi(wl[k]));
                hi[8 * v + 2 * k] = __float_as_uint(__uint_as_float(hi[8 * v + 2 * k]) * rs * bf16_lo(wh[k]));
                hi[8 * v + 2 * k + 1] = __float_as_uint(__uint_as_float(hi[8 * v + 2 * k + 1]) * rs * bf16_hi(wh[k]));
              }
            }
          }
          if (head < p.qkv.Hq + p.qkv.Hkv && row_ok) {
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              const float4 c2 = cs[i];   // (cos, sin) of frequencies 2i and 2i+1
              const float a0 = __uint_as_float(lo[2 * i]), b0 = __uint_as_float(hi[2 * i]);
              const float a1 = __uint_as_float(lo[2 * i + 1]), b1 = __uint_as_float(hi[2 * i + 1]);
              lo[2 * i] = __float_as_uint(a0 * c2.x - b0 * c2.y);
              hi[2 * i] = __float_as_uint(b0 * c2.x + a0 * c2.y);
              lo[2 * i + 1] = __float_as_uint(a1 * c2.z - b1 * c2.w);
              hi[2 * i + 1] = __float_as_uint(b1 * c2.z + a1 * c2.w);
            }
          }
          if (is_q) {
#pragma unroll
            for (int v = 0; v < 4; ++v) {
              *stg_chunk(buf, lane, v) = pack8(lo + 8 * v);
              *stg_chunk(buf, lane, 4 + v) = pack8(hi + 8 * v);
            }
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0 && live) {
              tma_store_2d(&tmC, buf, head * 64, wrow0);
              bulk_commit();
            }
            ++n_stores;
          } else if (row_ok && kv_ok) {
            // K and V rows go to the paged pool: one 128-byte line per (token, kv head)
            const bool is_k = head < p.qkv.Hq + p.qkv.Hkv;
            bf16* pool = is_k ? p.qkv.k_pool_layer : p.qkv.v_pool_layer;
            const int kvh = head - p.qkv.Hq - (is_k ? 0 : p.qkv.Hkv);
            uint4* d4 = reinterpret_cast<uint4*>(pool + (((size_t)blk * p.qkv.Hkv + kvh) * 64 + off) * 64);
#pragma unroll
            for (int v = 0; v < 4; ++v) {
              d4[v] = pack8(lo + 8 * v);
              d4[4 + v] = pack8(hi + 8 * v);
            }
          }
        }
      }
      else if (MODE == GS_QKV_ROPE128) {
        // head_dim 128: a head is 128 accumulator columns and the rotation pairs dim i with dim i + 64, so a head is
        // worked in two passes of 32 pairs (columns [32c, 32c+32) with [64+32c, 64+32c+32)); the row's (cos, sin) of
        // those 32 frequencies come from the table per pass.  q leaves through two staging buffers (dims 0..63 and
        // 64..127), both filled by the two passes and stored together.
        const bool kv_ok = live && phys >= 0 && phys < p.qkv.kv_rows;
        if (!kv_ok) phys = 0;
        const int blk = phys >> 6, off = phys & 63;
#pragma unroll 1
        for (int hh = 0; hh < BN / 128; ++hh) {
          const int head = n0 / 128 + hh;
          const bool is_q = head < p.qkv.Hq;
          const bool rot = head < p.qkv.Hq + p.qkv.Hkv;           // q and k heads are normalised (if asked) and rotated
          if (!slab_ok) break;
          float rs = 1.f;
          // (warp-uniform: a tensor-memory load is executed by the whole warp, rows beyond M included)
          const bool normed = p.qkv.q_norm && rot;
          if (normed) {                                            // per-head RMSNorm over the head's 128 dims
            float ss = 0.f;
#pragma unroll 1
            for (int c = 0; c < 4; ++c) {
              uint32_t r[32];
              tmem_ld32(t_acc + hh * 128 + c * 32, r);
              tmem_ld_wait();
#pragma unroll
              for (int i = 0; i < 32; ++i) ss += __uint_as_float(r[i]) * __uint_as_float(r[i]);
            }
            rs = rsqrtf(ss * (1.f / 128.f) + p.qkv.eps);
          }
          if (is_q) {
            if (lane == 0) bulk_wait_read<0>();                    // both staging buffers are free
            __syncwarp();
          }
          const bool is_k = rot && !is_q;
          bf16* pool = is_k ? p.qkv.k_pool_layer : p.qkv.v_pool_layer;
          const int kvh = head - p.qkv.Hq - (is_k || is_q ? 0 : p.qkv.Hkv);
          uint4* d4 = reinterpret_cast<uint4*>(pool + (((size_t)blk * p.qkv.Hkv + (is_q ? 0 : kvh)) * 64 + off) * 128);
#pragma unroll 1
          for (int c = 0; c < 2; ++c) {
            uint32_t lo[32], hi[32];
            tmem_ld32(t_acc + hh * 128 + c * 32, lo);
            tmem_ld32(t_acc + hh * 128 + 64 + c * 32, hi);
            tmem_ld_wait();
            if (normed && row_ok) {
              const uint4* g4 = reinterpret_cast<const uint4*>(is_q ? p.qkv.q_norm : p.qkv.k_norm);
#pragma unroll
              for (int v = 0; v < 4; ++v) {
                const uint4 gl = __ldg(g4 + 4 * c + v), gh = __ldg(g4 + 8 + 4 * c + v);
                const uint32_t wl[4] = {gl.x, gl.y, gl.z, gl.w}, wh[4] = {gh.x, gh.y, gh.z, gh.w};
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                  lo[8 * v + 2 * k] = __float_as_uint(__uint_as_float(lo[8 * v + 2 * k]) * rs * bf16_lo(wl[k]));
                  lo[8 * v + 2 * k + 1] = __float_as_uint(__uint_as_float(lo[8 * v + 2 * k + 1]) * rs * bf16_hi(wl[k]));
                  hi[8 * v + 2 * k] = __float_as_uint(__uint_as_float(hi[8 * v + 2 * k]) * rs * bf16_lo(wh[k]));
                  hi[8 * v + 2 * k + 1] = __float_as_uint(__uint_as_float(hi[8 * v + 2 * k + 1]) * rs * bf16_hi(wh[k]));
                }
              }
            }
            if (rot && row_ok) {
              const float4* src = reinterpret_cast<const float4*>(p.qkv.rope_cs + (size_t)row * 64 + c * 32);
#pragma unroll
              for (int i = 0; i < 16; ++i) {
                const float4 c2 = __ldg(src + i);   // (cos, sin) of frequencies 32c + 2i and 32c + 2i + 1
                const float a0 = __uint_as_float(lo[2 * i]), b0 = __uint_as_float(hi[2 * i]);
                const float a1 = __uint_as_float(lo[2 * i + 1]), b1 = __uint_as_float(hi[2 * i + 1]);
                lo[2 * i] = __float_as_uint(a0 * c2.x - b0 * c2.y);
                hi[2 * i] = __float_as_uint(b0 * c2.x + a0 * c2.y);
                lo[2 * i + 1] = __float_as_uint(a1 * c2.z - b1 * c2.w);
                hi[2 * i + 1] = __float_as_uint(b1 * c2.z + a1 * c2.w);
              }
            }
            if (is_q) {
#pragma unroll
              for (int v = 0; v < 4; ++v) {
                *stg_chunk(my_stg, lane, 4 * c + v) = pack8(lo + 8 * v);
                *stg_chunk(my_stg + STG_BYTES, lane, 4 * c + v) = pack8(hi + 8 * v);
              }
            } else if (row_ok && kv_ok) {
              // K and V rows go to the paged pool: one 256-byte row per (token, kv head)
#pragma unroll
              for (int v = 0; v < 4; ++v) {
                d4[4 * c + v] = pack8(lo + 8 * v);
                d4[8 + 4 * c + v] = pack8(hi + 8 * v);
              }
            }
          }
          if (is_q) {
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0 && live) {
              tma_store_2d(&tmC, my_stg, head * 128, wrow0);
              tma_store_2d(&tmC, my_stg + STG_BYTES, head * 128 + 64, wrow0);
              bulk_commit();
            }
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        if (PAIR) mbar_arrive_even_cta(tempty + b); else mbar_arrive(tempty + b);
      }
    }
    if (lane == 0) bulk_wait_all();               // staged rows have reached global memory (waiting only for the
                                                  // staging reads measured no shorter)
  }

done:
  tc_fence_before();
  __syncthreads();
  if (PAIR) cluster_sync();                // the other CTA's loads, MMAs and arrivals no longer touch this one
  if (warp == 1) {
    if (*abort_flag) __nanosleep(20000);   // let copies / MMAs in flight drain before TMEM goes away
    if (PAIR) tmem_dealloc_pair(tmem_base, C::TMEM_COLS); else tmem_dealloc(tmem_base, C::TMEM_COLS);
  }
}

// ------------------------------------------------------------------------------------------------
template <int BN, int MODE, bool PAIR>
static int launch_one(cudaStream_t st, const GemmSm100Args& a, int splits) {
  using C = Cfg<BN, PAIR>;
  constexpr int OUT_N = (MODE == GS_SWIGLU) ? BN / 2 : BN;
  static bool attr_set[kMaxDevices] = {};          // the attribute is per device
  if (a.device < 0 || a.device >= kMaxDevices) return -1;
  if (!attr_set[a.device]) {
    if (cudaFuncSetAttribute(gemm_sm100_kernel<BN, MODE, PAIR>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             C::SMEM_BYTES) != cudaSuccess)
      return -1;
    attr_set[a.device] = true;
  }
  GemmDev p;
  p.M = a.M;
  p.K = a.K;
  p.n_cols = (MODE == GS_SWIGLU) ? a.n_out / 2 : a.n_out;
  p.n_up_off = a.n_out / 2;
  const int k_blocks = a.K / BK;
  p.splits = splits;
  p.kb_per_split = (k_blocks + splits - 1) / splits;
  p.out = a.out;
  p.qkv = a.qkv;
  p.status = a.status;
  const int tile_m = PAIR ? 2 * BM : BM;
  const int m_tiles = (a.M + tile_m - 1) / tile_m;
  const int total = m_tiles * (p.n_cols / OUT_N) * splits;
  const int walkers = PAIR ? a.n_sms / 2 : a.n_sms;
  const int grid = (total < walkers ? total : walkers) * (PAIR ? 2 : 1);
  const CUtensorMap& tmB = a.tmB->m[PAIR ? 2 : (BN == 64 ? 0 : (BN == 128 ? 1 : 2))];   // pair: one 128-row box per CTA
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(kGemmThreads);
  cfg.dynamicSmemBytes = C::SMEM_BYTES;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  int n_attr = 0;
  if (a.pdl) {
    attr[n_attr].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[n_attr].val.programmaticStreamSerializationAllowed = 1;
    ++n_attr;
  }
  if (PAIR) {
    attr[n_attr].id = cudaLaunchAttributeClusterDimension;
    attr[n_attr].val.clusterDim.x = 2;
    attr[n_attr].val.clusterDim.y = 1;
    attr[n_attr].val.clusterDim.z = 1;
    ++n_attr;
  }
  cfg.attrs = attr;
  cfg.numAttrs = n_attr;
  return cudaLaunchKernelEx(&cfg, gemm_sm100_kernel<BN, MODE, PAIR>, a.tmA, tmB, a.tmC, p) == cudaSuccess ? 0 : -1;
}

// Tile width, CTA pairing and K slices: fewest cycles by a model calibrated on B200 (cycles per k-block of one work
// unit, measured in steady state with every SM busy: 128 x 256 tile ~820, 128 x 128 ~700, 128 x 64 ~600, CTA pair on
// 256 x 256 ~770 per CTA for twice the rows).  The 256-wide shapes run at the rate the whole chip's tensor pipes
// sustain (the measured library peak corresponds to ~730 cycles for such a k-block; one SM alone would need 544); the
// narrower ones are bound by L2 -> SM bytes.  A pair costs a cluster launch; the epilogue of the last unit of a CTA is
// exposed.
static void pick_tile(int mode, int n_cols, int M, int K, int n_sms, int max_splits, bool allow_pair, int* bn_out,
                      int* splits_out, bool* pair_out) {
  const int k_blocks = K / BK;
  const int cands[4] = {256, 256, 128, 64};     // first entry: a CTA pair on a 256 x 256 tile
  double best_cost = 1e30;
  *bn_out = (mode == GS_SWIGLU || mode == GS_QKV_ROPE128) ? 128 : 64;
  *splits_out = 1;
  *pair_out = false;
  for (int i = allow_pair ? 0 : 1; i < 4; ++i) {
    const bool pair = i == 0;
    const int bn = cands[i];
    const int out_n = (mode == GS_SWIGLU) ? bn / 2 : bn;
    if (n_cols % out_n || out_n % 64) continue;
    if (mode == GS_QKV_ROPE128 && bn < 128) continue;     // a tile holds whole 128-column heads
    const int tile_m = pair ? 2 * BM : BM;
    const int walkers = pair ? n_sms / 2 : n_sms;
    const long long tiles = (long long)((M + tile_m - 1) / tile_m) * (n_cols / out_n);
    for (int sp = 1; sp <= max_splits; ++sp) {
      const int kbs = (k_blocks + sp - 1) / sp;
      if (sp > 1 && (kbs < 4 || (long long)(sp - 1) * kbs >= k_blocks)) continue;
      const long long units = tiles * sp;
      const long long rounds = (units + walkers - 1) / walkers;
      const double per_kb = pair ? 770.0 : (bn == 256 ? 820.0 : (bn == 128 ? 700.0 : 600.0));
      const double epi = 700.0 + 10.0 * bn;
      const double cost = (double)rounds * (kbs * per_kb + 300.0) + epi + (sp > 1 ? 200.0 * sp : 0.0) + (pair ? 1500.0 : 0.0);
      if (cost < best_cost) { best_cost = cost; *bn_out = bn; *splits_out = sp; *pair_out = pair; }
    }
  }
}

template <int MODE>
static int launch_mode(cudaStream_t st, const GemmSm100Args& a) {
  const int n_cols = (MODE == GS_SWIGLU) ? a.n_out / 2 : a.n_out;
  int bn = 64, splits = 1;
  bool pair = false;
  pick_tile(MODE, n_cols, a.M, a.K, a.n_sms, (MODE == GS_ADD_F32 && a.max_splits > 1) ? a.max_splits : 1, a.pair != 0, &bn,
            &splits, &pair);
  if (a.force_bn) {
    const int fbn = a.force_bn == 512 ? 256 : a.force_bn;       // 512 = a CTA pair on 256-column tiles
    const int out_n = (MODE == GS_SWIGLU) ? fbn / 2 : fbn;
    if ((fbn != 64 && fbn != 128 && fbn != 256) || out_n % 64 || n_cols % out_n) return -1;
    if (MODE == GS_QKV_ROPE128 && fbn < 128) return -1;
    bn = fbn;
    pair = a.force_bn == 512;
  }
  if (a.force_splits) {
    const int kbs = (a.K / BK + a.force_splits - 1) / a.force_splits;
    if (MODE != GS_ADD_F32 || (a.force_splits - 1) * kbs >= a.K / BK) return -1;
    splits = a.force_splits;
  }
  if (pair) return launch_one<256, MODE, true>(st, a, splits);
  switch (bn) {
    case 256: return launch_one<256, MODE, false>(st, a, splits);
    case 128: return launch_one<128, MODE, false>(st, a, splits);
    default:
      if (MODE == GS_SWIGLU || MODE == GS_QKV_ROPE128) return launch_one<128, MODE, false>(st, a, splits);
      return launch_one<64, MODE, false>(st, a, splits);
  }
}

int launch_gemm_sm100(cudaStream_t st, const GemmSm100Args& a) {
  if (a.M <= 0) return 0;
  if (a.K % BK || a.n_out % 64 || !a.tmB) return -1;
  switch (a.mode) {
    case GS_STORE_BF16: return launch_mode<GS_STORE_BF16>(st, a);
    case GS_ADD_F32: return launch_mode<GS_ADD_F32>(st, a);
    case GS_SWIGLU: return launch_mode<GS_SWIGLU>(st, a);
    case GS_ARGMAX: return launch_mode<GS_ARGMAX>(st, a);
    case GS_QKV_ROPE: return launch_mode<GS_QKV_ROPE>(st, a);
    case GS_QKV_ROPE128: return launch_mode<GS_QKV_ROPE128>(st, a);
    default: return -1;
  }
}

}  // namespace hsd
