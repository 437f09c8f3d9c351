// tcgen05 / TMEM GEMM for sm_100a:  C = A W^T,  A [M,K] bf16 (activations), W [n_out,K] bf16 (weights),
// fp32 accumulation in tensor memory, operands staged in shared memory by TMA (128-byte swizzle).
//
// One persistent CTA per SM walks 128 x BN output tiles (M fastest, so CTAs running side by side share a
// weight tile through L2).  Warp roles: warp 0 = TMA producer (one elected lane), warp 1 = MMA issuer (one
// lane) and TMEM owner, warps 2..5 = epilogue (one TMEM lane quarter each).  Two accumulator buffers in
// TMEM let the epilogue of tile i overlap the main loop of tile i+1.
//
// Epilogues (all fused, nothing but the final result goes to HBM):
//   GS_STORE_BF16  C bf16 = acc
//   GS_ADD_F32     C fp32 += acc                         (O and down projections into the residual stream)
//   GS_SWIGLU      C bf16 = silu(gate) * up              (gate rows and up rows of W land in one tile)
//   GS_ARGMAX      per-row running argmax over the vocabulary + the next draft token's logit; logits never
//                  leave the SM (Eq. 10 of the paper fused into the LM head)
//   GS_QKV_ROPE    rotary embedding on q and k heads, q -> packed bf16, k/v -> paged KV pool
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

// ------------------------------------------------------------------------------------------------
constexpr int BM = 128;
constexpr int BK = 64;
constexpr int A_BYTES = BM * BK * 2;
constexpr int kGemmThreads = 192;

template <int BN>
struct Cfg {
  static constexpr int B_BYTES = BN * BK * 2;
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int STAGES = (BN == 256) ? 4 : (BN == 128 ? 6 : 8);
  static constexpr int TMEM_COLS = 2 * BN;
  static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/;
};

struct GemmDev {
  int M, n_cols, K, n_up_off;   // n_cols: output columns; n_up_off: row offset of the `up` half (SwiGLU)
  GemmOut out;
  QkvEpilogue qkv;
  int* status;
};

template <int BN, int MODE>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_sm100_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, GemmDev p) {
  using C = Cfg<BN>;
  constexpr int OUT_N = (MODE == GS_SWIGLU) ? BN / 2 : BN;   // output columns per tile
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + C::STAGES * C::STAGE_BYTES);
  uint64_t* full = bars;
  uint64_t* empty = bars + C::STAGES;
  uint64_t* tfull = bars + 2 * C::STAGES;
  uint64_t* tempty = tfull + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tempty + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < C::STAGES; ++s) {
      mbar_init(full + s, 1);
      mbar_init(empty + s, 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(tfull + b, 1);
      mbar_init(tempty + b, 4);
    }
    *abort_flag = 0;
    fence_mbar_init();
    tma_prefetch_desc(&tmA);
    tma_prefetch_desc(&tmB);
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, C::TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  const int m_tiles = (p.M + BM - 1) / BM;
  const int n_tiles = p.n_cols / OUT_N;
  const int total = m_tiles * n_tiles;
  const int k_blocks = p.K / BK;

  pdl_wait();

  if (warp == 0) {
    if (lane == 0) {
      int s = 0;
      uint32_t ph = 0;
      for (int t = blockIdx.x; t < total; t += gridDim.x) {
        const int m0 = (t % m_tiles) * BM, n0 = (t / m_tiles) * OUT_N;
        for (int kb = 0; kb < k_blocks; ++kb) {
          if (!mbar_wait(empty + s, ph ^ 1u, abort_flag, p.status, 100)) goto done;
          uint8_t* sa = smem + s * C::STAGE_BYTES;
          uint8_t* sb = sa + A_BYTES;
          mbar_expect_tx(full + s, C::STAGE_BYTES);
          tma_load_2d(sa, &tmA, full + s, kb * BK, m0);
          if (MODE == GS_SWIGLU) {
#pragma unroll
            for (int j = 0; j < OUT_N / 64; ++j) {
              tma_load_2d(sb + j * 8192, &tmB, full + s, kb * BK, n0 + j * 64);
              tma_load_2d(sb + (OUT_N / 64 + j) * 8192, &tmB, full + s, kb * BK, p.n_up_off + n0 + j * 64);
            }
          } else {
#pragma unroll
            for (int j = 0; j < BN / 64; ++j) tma_load_2d(sb + j * 8192, &tmB, full + s, kb * BK, n0 + j * 64);
          }
          if (++s == C::STAGES) { s = 0; ph ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc = umma_idesc_bf16(BN);
      int s = 0;
      uint32_t ph = 0;
      int it = 0;
      for (int t = blockIdx.x; t < total; t += gridDim.x, ++it) {
        const int b = it & 1;
        const uint32_t aph = (it >> 1) & 1;
        if (!mbar_wait(tempty + b, aph ^ 1u, abort_flag, p.status, 200)) goto done;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + b * BN;
        for (int kb = 0; kb < k_blocks; ++kb) {
          if (!mbar_wait(full + s, ph, abort_flag, p.status, 201)) goto done;
          tc_fence_after();
          const uint32_t sa = smem_u32(smem + s * C::STAGE_BYTES);
          const uint32_t sb = sa + A_BYTES;
#pragma unroll
          for (int k = 0; k < BK / 16; ++k) {
            umma_bf16(d_tmem, umma_desc_sw128(sa + k * 32), umma_desc_sw128(sb + k * 32), idesc, (kb | k) != 0);
          }
          umma_commit(empty + s);      // smem stage reusable once these MMAs have read it
          if (++s == C::STAGES) { s = 0; ph ^= 1u; }
        }
        umma_commit(tfull + b);        // accumulator complete
      }
    }
  } else {
    const int quarter = warp & 3;                 // TMEM lanes [32*quarter, +32) belong to this warp
    const int row_in_tile = quarter * 32 + lane;
    int it = 0;
    for (int t = blockIdx.x; t < total; t += gridDim.x, ++it) {
      const int b = it & 1;
      const uint32_t aph = (it >> 1) & 1;
      const int m0 = (t % m_tiles) * BM, n0 = (t / m_tiles) * OUT_N;
      const int row = m0 + row_in_tile;
      const bool row_ok = row < p.M;
      bool ok = mbar_wait(tfull + b, aph, abort_flag, p.status, 300);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) goto done;
      tc_fence_after();
      const uint32_t t_acc = tmem_base + (uint32_t(quarter * 32) << 16) + b * BN;

      if (MODE == GS_STORE_BF16 || MODE == GS_ADD_F32) {
#pragma unroll 1
        for (int c = 0; c < BN; c += 32) {
          uint32_t r[32];
          tmem_ld32(t_acc + c, r);
          tmem_ld_wait();
          if (row_ok) {
            if (MODE == GS_STORE_BF16) {
              uint4* dst = reinterpret_cast<uint4*>(reinterpret_cast<bf16*>(p.out.C) + (size_t)row * p.out.ldc + n0 + c);
#pragma unroll
              for (int v = 0; v < 4; ++v) {
                uint4 o;
                o.x = pack_bf16(__uint_as_float(r[8 * v + 0]), __uint_as_float(r[8 * v + 1]));
                o.y = pack_bf16(__uint_as_float(r[8 * v + 2]), __uint_as_float(r[8 * v + 3]));
                o.z = pack_bf16(__uint_as_float(r[8 * v + 4]), __uint_as_float(r[8 * v + 5]));
                o.w = pack_bf16(__uint_as_float(r[8 * v + 6]), __uint_as_float(r[8 * v + 7]));
                dst[v] = o;
              }
            } else {
              float4* dst = reinterpret_cast<float4*>(reinterpret_cast<float*>(p.out.C) + (size_t)row * p.out.ldc + n0 + c);
#pragma unroll
              for (int v = 0; v < 8; ++v) {
                float4 o = dst[v];
                o.x += __uint_as_float(r[4 * v + 0]);
                o.y += __uint_as_float(r[4 * v + 1]);
                o.z += __uint_as_float(r[4 * v + 2]);
                o.w += __uint_as_float(r[4 * v + 3]);
                dst[v] = o;
              }
            }
          }
        }
      } else if (MODE == GS_SWIGLU) {
#pragma unroll 1
        for (int c = 0; c < OUT_N; c += 32) {
          uint32_t g[32], u[32];
          tmem_ld32(t_acc + c, g);
          tmem_ld32(t_acc + OUT_N + c, u);
          tmem_ld_wait();
          if (row_ok) {
            uint4* dst = reinterpret_cast<uint4*>(reinterpret_cast<bf16*>(p.out.C) + (size_t)row * p.out.ldc + n0 + c);
#pragma unroll
            for (int v = 0; v < 4; ++v) {
              float o[8];
#pragma unroll
              for (int e = 0; e < 8; ++e) {
                const float gv = __uint_as_float(g[8 * v + e]);
                o[e] = gv / (1.f + __expf(-gv)) * __uint_as_float(u[8 * v + e]);
              }
              uint4 w;
              w.x = pack_bf16(o[0], o[1]);
              w.y = pack_bf16(o[2], o[3]);
              w.z = pack_bf16(o[4], o[5]);
              w.w = pack_bf16(o[6], o[7]);
              dst[v] = w;
            }
          }
        }
      } else if (MODE == GS_ARGMAX) {
        const int nxt = (row_ok && p.out.row_next) ? p.out.row_next[row] : -1;
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
        const int phys = row_ok ? p.qkv.row_kv[row] : 0;
        const int blk = phys >> 6, off = phys & 63;
#pragma unroll 1
        for (int hh = 0; hh < BN / 64; ++hh) {
          uint32_t lo[32], hi[32];
          tmem_ld32(t_acc + hh * 64, lo);
          tmem_ld32(t_acc + hh * 64 + 32, hi);
          tmem_ld_wait();
          if (!row_ok) continue;
          const int head = n0 / 64 + hh;
          if (head < p.qkv.Hq + p.qkv.Hkv) {
            const float4* cs = reinterpret_cast<const float4*>(p.qkv.rope_cs + (size_t)row * 32);
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
            bf16* dst = (head < p.qkv.Hq)
                            ? p.qkv.q_out + (size_t)row * p.qkv.Hq * 64 + head * 64
                            : p.qkv.k_pool_layer + (((size_t)blk * p.qkv.Hkv + (head - p.qkv.Hq)) * 64 + off) * 64;
            uint4* d4 = reinterpret_cast<uint4*>(dst);
#pragma unroll
            for (int v = 0; v < 4; ++v) {
              uint4 o;
              o.x = pack_bf16(__uint_as_float(lo[8 * v + 0]), __uint_as_float(lo[8 * v + 1]));
              o.y = pack_bf16(__uint_as_float(lo[8 * v + 2]), __uint_as_float(lo[8 * v + 3]));
              o.z = pack_bf16(__uint_as_float(lo[8 * v + 4]), __uint_as_float(lo[8 * v + 5]));
              o.w = pack_bf16(__uint_as_float(lo[8 * v + 6]), __uint_as_float(lo[8 * v + 7]));
              d4[v] = o;
              uint4 q;
              q.x = pack_bf16(__uint_as_float(hi[8 * v + 0]), __uint_as_float(hi[8 * v + 1]));
              q.y = pack_bf16(__uint_as_float(hi[8 * v + 2]), __uint_as_float(hi[8 * v + 3]));
              q.z = pack_bf16(__uint_as_float(hi[8 * v + 4]), __uint_as_float(hi[8 * v + 5]));
              q.w = pack_bf16(__uint_as_float(hi[8 * v + 6]), __uint_as_float(hi[8 * v + 7]));
              d4[4 + v] = q;
            }
          } else {
            // V is stored transposed per block: [dim][token]; consecutive lanes hold consecutive tokens
            bf16* dst = p.qkv.v_pool_layer + ((size_t)blk * p.qkv.Hkv + (head - p.qkv.Hq - p.qkv.Hkv)) * 4096 + off;
#pragma unroll
            for (int e = 0; e < 32; ++e) {
              dst[(size_t)e * 64] = __float2bfloat16(__uint_as_float(lo[e]));
              dst[(size_t)(e + 32) * 64] = __float2bfloat16(__uint_as_float(hi[e]));
            }
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(tempty + b);
    }
  }

done:
  pdl_launch_dependents();
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    if (*abort_flag) __nanosleep(20000);   // let copies / MMAs in flight drain before TMEM goes away
    tmem_dealloc(tmem_base, C::TMEM_COLS);
  }
}

// ------------------------------------------------------------------------------------------------
template <int BN, int MODE>
static int launch_one(cudaStream_t st, const GemmSm100Args& a, int out_n_per_tile) {
  using C = Cfg<BN>;
  static bool attr_set = false;
  if (!attr_set) {
    if (cudaFuncSetAttribute(gemm_sm100_kernel<BN, MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES) !=
        cudaSuccess)
      return -1;
    attr_set = true;
  }
  GemmDev p;
  p.M = a.M;
  p.K = a.K;
  p.n_cols = (MODE == GS_SWIGLU) ? a.n_out / 2 : a.n_out;
  p.n_up_off = a.n_out / 2;
  p.out = a.out;
  p.qkv = a.qkv;
  p.status = a.status;
  const int m_tiles = (a.M + BM - 1) / BM;
  const int total = m_tiles * (p.n_cols / out_n_per_tile);
  const int grid = total < a.n_sms ? total : a.n_sms;
  gemm_sm100_kernel<BN, MODE><<<grid, kGemmThreads, C::SMEM_BYTES, st>>>(a.tmA, a.tmB, p);
  return cudaGetLastError() == cudaSuccess ? 0 : -1;
}

// Tile width: fewest (waves x per-tile time), narrow tiles discounted for their lower MMA efficiency.
static int pick_bn(int mode, int n_cols, int M, int n_sms) {
  const int m_tiles = (M + BM - 1) / BM;
  const int cands[3] = {256, 128, 64};
  const double eff[3] = {1.0, 0.9, 0.6};
  int best = (mode == GS_SWIGLU) ? 128 : 64;
  double best_cost = 1e30;
  for (int i = 0; i < 3; ++i) {
    const int bn = cands[i];
    const int out_n = (mode == GS_SWIGLU) ? bn / 2 : bn;
    if (n_cols % out_n || out_n % 64) continue;   // B rows arrive in 64-row TMA boxes
    const long long tiles = (long long)m_tiles * (n_cols / out_n);
    const long long waves = (tiles + n_sms - 1) / n_sms;
    const double cost = (double)waves * bn / eff[i];
    if (cost < best_cost) { best_cost = cost; best = bn; }
  }
  return best;
}

int gemm_sm100_box_rows(int, int, int, int) { return 64; }

template <int MODE>
static int launch_mode(cudaStream_t st, const GemmSm100Args& a) {
  const int n_cols = (MODE == GS_SWIGLU) ? a.n_out / 2 : a.n_out;
  const int bn = pick_bn(MODE, n_cols, a.M, a.n_sms);
  switch (bn) {
    case 256: return launch_one<256, MODE>(st, a, MODE == GS_SWIGLU ? 128 : 256);
    case 128: return launch_one<128, MODE>(st, a, MODE == GS_SWIGLU ? 64 : 128);
    default:
      if (MODE == GS_SWIGLU) return launch_one<128, MODE>(st, a, 64);
      return launch_one<64, MODE>(st, a, 64);
  }
}

int launch_gemm_sm100(cudaStream_t st, const GemmSm100Args& a) {
  if (a.M <= 0) return 0;
  if (a.K % BK || a.n_out % 64) return -1;
  switch (a.mode) {
    case GS_STORE_BF16: return launch_mode<GS_STORE_BF16>(st, a);
    case GS_ADD_F32: return launch_mode<GS_ADD_F32>(st, a);
    case GS_SWIGLU: return launch_mode<GS_SWIGLU>(st, a);
    case GS_ARGMAX: return launch_mode<GS_ARGMAX>(st, a);
    case GS_QKV_ROPE: return launch_mode<GS_QKV_ROPE>(st, a);
    default: return -1;
  }
}

}  // namespace hsd
