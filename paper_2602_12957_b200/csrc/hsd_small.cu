// Memory- and latency-bound kernels of the verify step: row metadata + checks, embedding gather,
// RMSNorm, RoPE + paged KV write, the plain SIMT attention (debug cross-check), accept/emit, KV commit.
#include "hsd_kernels.h"

namespace hsd {

const char* kernel_class_name(int kc) {
  static const char* names[KC_COUNT] = {"setup_rows", "embed",     "rmsnorm",     "gemm_qkv",  "rope_kv_write",
                                        "attention",  "attn_combine", "gemm_o",   "gemm_gate_up", "gemm_down",
                                        "lm_head_argmax", "accept_emit", "kv_commit", "debug"};
  return (kc >= 0 && kc < KC_COUNT) ? names[kc] : "?";
}

// ------------------------------------------------------------------------------------------------
// Row metadata.  One CTA per sequence.  Validates what the host cannot see (device-resident lengths and
// tables); any violation sets the status words, and every kernel that follows an indirection returns early.
constexpr int kSetupRows = 64;   // rows of one sequence handled by one CTA
__global__ void setup_rows_kernel(SetupArgs a, KvView kv, RowMeta rm, int* status, int* tile_count) {
  pdl_wait();               // everything below reads or writes what earlier kernels of the step produced
  pdl_launch_dependents();
  const int i = blockIdx.x;
  const int tid = threadIdx.x;
  __shared__ int s_red[32];
  __shared__ int s_bad;
  if (tid == 0) s_bad = 0;
  __syncthreads();

  // every CTA scans cu_q once: monotone + total, and the exclusive scan of q-tiles before sequence i
  int my_tiles = 0, bad = 0;
  for (int s = tid; s < a.n_seqs; s += blockDim.x) {
    const int n = a.cu_q[s + 1] - a.cu_q[s];
    if (n < 0) bad = 1;
    if (n > a.max_q_len) bad = 2;
    if (s < i && n > 0) my_tiles += (n + a.tokens_per_tile - 1) / a.tokens_per_tile;
  }
  if (tid == 0 && (a.cu_q[0] != 0 || a.cu_q[a.n_seqs] != a.total_q)) bad = 1;
  for (int o = 16; o; o >>= 1) my_tiles += __shfl_xor_sync(0xffffffffu, my_tiles, o);
  if ((tid & 31) == 0) s_red[tid >> 5] = my_tiles;
  if (bad) atomicMax(&s_bad, bad);
  __syncthreads();
  int tile0 = 0;
  for (int w = 0; w < (blockDim.x >> 5); ++w) tile0 += s_red[w];
  if (s_bad) {
    if (tid == 0 && blockIdx.y == 0) dev_fail(status, s_bad == 2 ? DEV_TOO_LONG : DEV_CU_Q, i);
    return;
  }

  const int q0 = a.cu_q[i];
  const int n = a.cu_q[i + 1] - q0;
  const int slot = a.seq_slots ? a.seq_slots[i] : a.slot_base + i;
  if (slot < 0 || slot >= kv.n_slots) {
    if (tid == 0) dev_fail(status, DEV_KV_CAPACITY, i);
    return;
  }
  const int L = kv.seq_lens[slot];
  if (L < 0 || (long long)L + n > (long long)kv.max_blocks * HSD_KV_BLOCK) {
    if (tid == 0) dev_fail(status, DEV_KV_CAPACITY, i);
    return;
  }
  if (tid == 0 && blockIdx.y == 0) {
    rm.seq_q0[i] = q0;
    rm.seq_n[i] = n;
    rm.seq_len[i] = L;
    rm.seq_slot[i] = slot;
    rm.seq_tile0[i] = tile0;
    if (i == a.n_seqs - 1) {
      const int t = tile0 + (n + a.tokens_per_tile - 1) / a.tokens_per_tile;
      rm.seq_tile0[a.n_seqs] = t;
      *tile_count = t;
    }
  }
  const int j_lo = blockIdx.y * kSetupRows;
  const int j_hi = min(n, j_lo + kSetupRows);
  const int half = a.head_dim / 2;
  // Candidate tree: a row's rotary position is its depth below the pending token, not its index in the call
  // (Sec. 3.2: a node continues the path pi(v), whatever else is packed beside it).
  __shared__ int s_depth[kSetupRows];
  if (a.parent) {
    for (int j = j_lo + tid; j < j_hi; j += blockDim.x) {
      uint32_t m[4] = {0u, 0u, 0u, 0u};
      int d = 0, pj = j;
      bool ok = j < 128;
      if (ok) m[j >> 5] |= 1u << (j & 31);
      if (j > 0 && a.parent[q0 + j] == -2) pj = 0;      // padding row: no parent, no children, sees only itself
      while (ok && pj > 0) {
        const int pp = a.parent[q0 + pj];
        if (pp < 0 || pp >= pj) { ok = false; break; }
        pj = pp;
        m[pj >> 5] |= 1u << (pj & 31);
        ++d;
      }
      if (j == 0 && a.parent[q0] != -1) ok = false;
      if (!ok) {
        dev_fail(status, DEV_TREE, q0 + j);
        d = 0;
      }
      s_depth[j - j_lo] = d;
      const int r = q0 + j;
      rm.anc[r] = make_uint4(m[0], m[1], m[2], m[3]);
      rm.lm_src[r] = r;
      rm.lm_next[r] = -1;
      const bool child = ok && j > 0 && a.parent[r] >= 0;
      rm.lm_src[a.total_q + r] = child ? q0 + a.parent[r] : r;
      rm.lm_next[a.total_q + r] = child ? a.tokens[r] : -1;
    }
    __syncthreads();
  }
  for (int j = j_lo + tid; j < j_hi; j += blockDim.x) {
    const int r = q0 + j;
    int tok, nxt = -1;
    if (a.tokens) {
      tok = a.tokens[r];
      if (j + 1 < n) nxt = a.tokens[r + 1];
    } else {
      tok = (j == 0) ? a.pending[0] : a.draft[j - 1];
      if (j + 1 < n) nxt = a.draft[j];
    }
    if (tok >= a.vocab || (tok < 0 && !a.allow_embed_rows)) {
      dev_fail(status, DEV_TOKEN_RANGE, r);
      tok = 0;
    }
    if (tok < 0) tok = -1;
    const int pos = L + j;
    int phys = kv.block_table[(size_t)slot * kv.max_blocks + pos / HSD_KV_BLOCK];
    if (phys < 0 || phys >= kv.n_blocks) {
      dev_fail(status, DEV_BLOCK_RANGE, r);
      phys = 0;
    }
    rm.row_seq[r] = i;
    rm.row_pos[r] = a.parent ? L + s_depth[j - j_lo] : pos;
    rm.row_tok[r] = tok;
    rm.row_kv[r] = phys * HSD_KV_BLOCK + pos % HSD_KV_BLOCK;
    rm.row_next[r] = (a.allow_embed_rows || a.parent) ? -1 : nxt;
  }
  // rotary table: (cos, sin) of pos * base^(-2i/D), angle formed in double so long contexts keep accuracy
  for (int e = j_lo * half + tid; e < j_hi * half; e += blockDim.x) {
    const int j = e / half, f = e % half;
    const double inv = exp2(-(double)(2 * f) / (double)a.head_dim * log2((double)a.rope_base));
    double sn, cs;
    sincos((double)(L + (a.parent ? s_depth[j - j_lo] : j)) * inv, &sn, &cs);
    rm.rope_cs[(size_t)(q0 + j) * half + f] = make_float2((float)cs, (float)sn);
  }
}

void launch_setup_rows(cudaStream_t st, const SetupArgs& a, const KvView& kv, const RowMeta& rm, int* status,
                       int* tile_count, bool pdl) {
  dim3 grid(a.n_seqs, (a.max_q_len + kSetupRows - 1) / kSetupRows);
  launch_kernel(setup_rows_kernel, grid, dim3(256), 0, st, pdl, a, kv, rm, status, tile_count);
}

// ------------------------------------------------------------------------------------------------
// Embedding gather: x[r] = fp32(table[tok]) or fp32(embeds[r]).  One warp per row, 16-byte loads.
__global__ void embed_kernel(RowMeta rm, const bf16* __restrict__ table, const bf16* __restrict__ embeds,
                             float* __restrict__ x, int T, int d, const int* status) {
  pdl_wait();               // everything below reads or writes what earlier kernels of the step produced
  pdl_launch_dependents();
  if (*status) return;
  const int r = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (r >= T) return;
  const int lane = threadIdx.x & 31;
  const int tok = rm.row_tok[r];
  const bf16* src = tok >= 0 ? table + (size_t)tok * d : embeds + (size_t)r * d;
  float* dst = x + (size_t)r * d;
  for (int c = lane * 8; c < d; c += 256) {
    uint4 v = *reinterpret_cast<const uint4*>(src + c);
    float4 lo = make_float4(bf16_lo(v.x), bf16_hi(v.x), bf16_lo(v.y), bf16_hi(v.y));
    float4 hi = make_float4(bf16_lo(v.z), bf16_hi(v.z), bf16_lo(v.w), bf16_hi(v.w));
    *reinterpret_cast<float4*>(dst + c) = lo;
    *reinterpret_cast<float4*>(dst + c + 4) = hi;
  }
}
void launch_embed(cudaStream_t st, const RowMeta& rm, const bf16* table, const bf16* embeds, float* x, int T, int d,
                  const int* status, bool pdl) {
  launch_kernel(embed_kernel, dim3((T + 7) / 8), dim3(256), 0, st, pdl, rm, table, embeds, x, T, d, status);
}

// ------------------------------------------------------------------------------------------------
// RMSNorm: h = bf16(x * rsqrt(mean(x^2) + eps) * gain).  One warp per row; the row stays in registers
// between the reduction and the scaling (d <= 4096), so x is read once.
template <int VEC>   // VEC float4 per lane: d = 128 * VEC
__global__ void rmsnorm_kernel(const float* __restrict__ x, const bf16* __restrict__ gain, bf16* __restrict__ h,
                               int rows, int d, float eps, const int* __restrict__ sel_rows, int src_rows,
                               const int* __restrict__ status) {
  pdl_wait();               // everything below reads or writes what earlier kernels of the step produced
  pdl_launch_dependents();
  const int r = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (r >= rows) return;
  const int lane = threadIdx.x & 31;
  // the gather form follows an index an earlier kernel of the step wrote: after a failed device-side check that
  // index was never written, so nothing is read through it (and an index outside the source is never followed)
  if (sel_rows && status && *status) return;
  const int src = sel_rows ? sel_rows[r] : r;
  if (src < 0 || src >= src_rows) return;
  const float4* xp = reinterpret_cast<const float4*>(x + (size_t)src * d);
  const uint2* gp = reinterpret_cast<const uint2*>(gain);
  float4 v[VEC];
  uint2 gv[VEC];
#pragma unroll
  for (int i = 0; i < VEC; ++i) v[i] = xp[lane + 32 * i];
#pragma unroll
  for (int i = 0; i < VEC; ++i) gv[i] = __ldg(gp + lane + 32 * i);      // in flight together with the row
  float ss = 0.f;
#pragma unroll
  for (int i = 0; i < VEC; ++i) ss += v[i].x * v[i].x + v[i].y * v[i].y + v[i].z * v[i].z + v[i].w * v[i].w;
  for (int o = 16; o; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
  const float rs = rsqrtf(ss / (float)d + eps);
  uint2* hp = reinterpret_cast<uint2*>(h + (size_t)r * d);
#pragma unroll
  for (int i = 0; i < VEC; ++i) {
    const uint2 g = gv[i];
    uint2 o;
    o.x = pack_bf16(v[i].x * rs * bf16_lo(g.x), v[i].y * rs * bf16_hi(g.x));
    o.y = pack_bf16(v[i].z * rs * bf16_lo(g.y), v[i].w * rs * bf16_hi(g.y));
    hp[lane + 32 * i] = o;
  }
}
void launch_rmsnorm(cudaStream_t st, const float* x, const bf16* gain, bf16* h, int rows, int d, float eps,
                    const int* sel_rows, int src_rows, const int* status, bool pdl) {
  if (rows <= 0) return;
  dim3 grid((rows + 7) / 8), block(256);
#define HSD_RMS_CASE(V) \
  case V: launch_kernel(rmsnorm_kernel<V>, grid, block, 0, st, pdl, x, gain, h, rows, d, eps, sel_rows, src_rows, status); break;
  switch (d / 128) {
    HSD_RMS_CASE(1) HSD_RMS_CASE(2) HSD_RMS_CASE(4) HSD_RMS_CASE(8) HSD_RMS_CASE(16) HSD_RMS_CASE(32)
    default: break;   // hsd_create rejects other widths
  }
#undef HSD_RMS_CASE
}

__global__ void select_last_rows_kernel(RowMeta rm, int n_seqs, int* sel_rows, const int* status) {
  pdl_wait();               // everything below reads or writes what earlier kernels of the step produced
  pdl_launch_dependents();
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n_seqs) return;
  // after a failed check the per-sequence metadata was not written: name no row at all
  sel_rows[i] = *status ? -1 : rm.seq_q0[i] + max(rm.seq_n[i], 1) - 1;
}
void launch_select_last_rows(cudaStream_t st, const RowMeta& rm, int n_seqs, int* sel_rows, const int* status, bool pdl) {
  launch_kernel(select_last_rows_kernel, dim3((n_seqs + 127) / 128), dim3(128), 0, st, pdl, rm, n_seqs, sel_rows, status);
}

__global__ void clear_best_kernel(unsigned long long* row_best, float* zdraft, int rows) {
  pdl_wait();               // everything below reads or writes what earlier kernels of the step produced
  pdl_launch_dependents();
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < rows) {
    row_best[i] = 0ull;
    if (zdraft) zdraft[i] = __int_as_float(0x7fc00000);
  }
}
void launch_clear_best(cudaStream_t st, unsigned long long* row_best, float* zdraft, int rows, bool pdl) {
  launch_kernel(clear_best_kernel, dim3((rows + 255) / 256), dim3(256), 0, st, pdl, row_best, zdraft, rows);
}

__global__ void unpack_best_kernel(const unsigned long long* row_best, int rows, int* argmax, float* zmax) {
  pdl_wait();               // everything below reads or writes what earlier kernels of the step produced
  pdl_launch_dependents();
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < rows) {
    const unsigned long long b = row_best[i];
    if (argmax) argmax[i] = key_col(b);
    if (zmax) zmax[i] = key_value(b);
  }
}
void launch_unpack_best(cudaStream_t st, const unsigned long long* row_best, int rows, int* argmax, float* zmax,
                        bool pdl) {
  launch_kernel(unpack_best_kernel, dim3((rows + 255) / 256), dim3(256), 0, st, pdl, row_best, rows, argmax, zmax);
}

// ------------------------------------------------------------------------------------------------
// RoPE + paged KV write from an fp32 qkv row (SIMT path; the tensor-core path fuses this into the
// QKV projection's epilogue).  One warp per (row, head); lane i holds dims i and i + 32.
__global__ void rope_kvwrite_kernel(const float* __restrict__ qkv, RowMeta rm, KvView kv, ModelDims md, int layer,
                                    bf16* __restrict__ q, int T, const int* status, const bf16* __restrict__ q_norm,
                                    const bf16* __restrict__ k_norm) {
  if (*status) return;
  const int heads = md.Hq + 2 * md.Hkv;
  const int w = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (w >= T * heads) return;
  const int r = w / heads, hd = w % heads, lane = threadIdx.x & 31;
  const float* src = qkv + (size_t)r * md.qkv_out + hd * 64;
  float a = src[lane], b = src[lane + 32];
  const int phys = rm.row_kv[r];
  const size_t blk_base = ((size_t)layer * kv.n_blocks + phys / 64) * md.Hkv;
  const int off = phys % 64;
  if (hd < md.Hq + md.Hkv) {
    if (q_norm) {       // per-head RMSNorm over the 64 dims before the rotation
      float ss = a * a + b * b;
      for (int o = 16; o; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
      const float rs = rsqrtf(ss * (1.f / 64.f) + md.eps);
      const bf16* g = hd < md.Hq ? q_norm : k_norm;
      a *= rs * __bfloat162float(g[lane]);
      b *= rs * __bfloat162float(g[lane + 32]);
    }
    const float2 cs = rm.rope_cs[(size_t)r * 32 + lane];
    const float ra = a * cs.x - b * cs.y, rb = b * cs.x + a * cs.y;
    if (hd < md.Hq) {
      bf16* dst = q + (size_t)r * md.Hq * 64 + hd * 64;
      dst[lane] = __float2bfloat16(ra);
      dst[lane + 32] = __float2bfloat16(rb);
    } else {
      bf16* dst = kv.k_pool + ((blk_base + (hd - md.Hq)) * 64 + off) * 64;
      dst[lane] = __float2bfloat16(ra);
      dst[lane + 32] = __float2bfloat16(rb);
    }
  } else {
    bf16* dst = kv.v_pool + ((blk_base + (hd - md.Hq - md.Hkv)) * 64 + off) * 64;
    dst[lane] = __float2bfloat16(a);
    dst[lane + 32] = __float2bfloat16(b);
  }
}
void launch_rope_kvwrite(cudaStream_t st, const float* qkv, const RowMeta& rm, const KvView& kv, const ModelDims& md,
                         int layer, bf16* q, int T, const int* status, const bf16* q_norm, const bf16* k_norm) {
  const long long warps = (long long)T * (md.Hq + 2 * md.Hkv);
  rope_kvwrite_kernel<<<(unsigned)((warps + 7) / 8), 256, 0, st>>>(qkv, rm, kv, md, layer, q, T, status, q_norm, k_norm);
}

// ------------------------------------------------------------------------------------------------
// Plain SIMT attention (debug cross-check): one warp per (row, q head), online softmax over 32-key chunks.
__global__ void attn_simt_kernel(const bf16* __restrict__ q, RowMeta rm, KvView kv, ModelDims md, int layer,
                                 bf16* __restrict__ out, int T, const int* status) {
  if (*status) return;
  const int w = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (w >= T * md.Hq) return;
  const int r = w / md.Hq, hq = w % md.Hq, lane = threadIdx.x & 31;
  const int kvh = hq / md.group;
  const int seq = rm.row_seq[r];
  const int slot = rm.seq_slot[seq];
  const int n_keys = rm.row_pos[r] + 1;            // keys at positions 0 .. pos (causal, own row included)
  __shared__ float s_q[8][64];
  float* qs = s_q[threadIdx.x >> 5];
  const bf16* qp = q + (size_t)r * md.Hq * 64 + hq * 64;
  qs[lane] = __bfloat162float(qp[lane]) * 0.125f;   // 1/sqrt(64)
  qs[lane + 32] = __bfloat162float(qp[lane + 32]) * 0.125f;
  __syncwarp();
  float m = -INFINITY, l = 0.f, o0 = 0.f, o1 = 0.f;
  const int* bt = kv.block_table + (size_t)slot * kv.max_blocks;
  for (int k0 = 0; k0 < n_keys; k0 += 32) {
    const int key = k0 + lane;
    const int phys = bt[k0 / 64];                   // a 32-key chunk never straddles a 64-token block
    const size_t tile = ((size_t)layer * kv.n_blocks + phys) * md.Hkv + kvh;
    float s = -INFINITY;
    if (key < n_keys) {
      const uint4* kp = reinterpret_cast<const uint4*>(kv.k_pool + (tile * 64 + key % 64) * 64);
      float acc = 0.f;
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        uint4 v = kp[c];
        const float* qq = qs + c * 8;
        acc += qq[0] * bf16_lo(v.x) + qq[1] * bf16_hi(v.x) + qq[2] * bf16_lo(v.y) + qq[3] * bf16_hi(v.y) +
               qq[4] * bf16_lo(v.z) + qq[5] * bf16_hi(v.z) + qq[6] * bf16_lo(v.w) + qq[7] * bf16_hi(v.w);
      }
      s = acc;
    }
    float cm = s;
    for (int o = 16; o; o >>= 1) cm = fmaxf(cm, __shfl_xor_sync(0xffffffffu, cm, o));
    const float m_new = fmaxf(m, cm);
    const float p = (key < n_keys) ? __expf(s - m_new) : 0.f;
    float ps = p;
    for (int o = 16; o; o >>= 1) ps += __shfl_xor_sync(0xffffffffu, ps, o);
    const float scale = __expf(m - m_new);
    l = l * scale + ps;
    o0 *= scale;
    o1 *= scale;
    m = m_new;
    // V tile [tok][dim]: lane owns dims lane and lane + 32
    const bf16* vt = kv.v_pool + tile * 4096;
    const int tok0 = k0 % 64;
    const int cnt = min(32, n_keys - k0);
    for (int t = 0; t < cnt; ++t) {
      const float pt = __shfl_sync(0xffffffffu, p, t);
      o0 += pt * __bfloat162float(vt[(size_t)(tok0 + t) * 64 + lane]);
      o1 += pt * __bfloat162float(vt[(size_t)(tok0 + t) * 64 + lane + 32]);
    }
  }
  bf16* op = out + (size_t)r * md.Hq * 64 + hq * 64;
  op[lane] = __float2bfloat16(o0 / l);
  op[lane + 32] = __float2bfloat16(o1 / l);
}
void launch_attn_simt(cudaStream_t st, const bf16* q, const RowMeta& rm, const KvView& kv, const ModelDims& md,
                      int layer, bf16* out, int T, const int* status) {
  const long long warps = (long long)T * md.Hq;
  attn_simt_kernel<<<(unsigned)((warps + 7) / 8), 256, 0, st>>>(q, rm, kv, md, layer, out, T, status);
}

// ------------------------------------------------------------------------------------------------
// Draft compare + longest-prefix accept + emit.  One warp per sequence.
// Row j (0-based) of a sequence holds the distribution after [.., pending, d_1..d_j]; its next draft token is
// d_{j+1}.  a = first j < k whose test fails (or k).  Exact mode: argmax == d_{j+1}.  Threshold mode:
// z[d_{j+1}] - z_max >= log_tau.
__global__ void accept_kernel(AcceptArgs a, RowMeta rm, const int* status) {
  pdl_wait();               // everything below reads or writes what earlier kernels of the step produced
  pdl_launch_dependents();
  const int i = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (i >= a.n_seqs) return;
  const int lane = threadIdx.x & 31;
  // (three independent reads in flight together; after a failed check the two row words are unwritten and unused)
  const int failed = *status;
  const int q0 = rm.seq_q0[i], n = rm.seq_n[i];
  if (failed) {             // a failed step decides nothing: -1 makes the commit that follows leave the lengths alone
    if (lane == 0) { a.accept_len[i] = -1; a.n_emit[i] = 0; }
    return;
  }
  if (n <= 0) {
    if (lane == 0) { a.accept_len[i] = 0; a.n_emit[i] = 0; }
    return;
  }
  const int k = n - 1;
  int acc = k;
  for (int j0 = 0; j0 < k && acc == k; j0 += 32) {
    const int j = j0 + lane;
    bool ok = true;
    if (j < k) {
      const unsigned long long best = a.row_best[q0 + j];
      const int nxt = rm.row_next[q0 + j];
      if (a.log_tau == 0.f) ok = (key_col(best) == nxt);
      else ok = (a.zdraft[q0 + j] - key_value(best) >= a.log_tau);
    }
    const unsigned fail = __ballot_sync(0xffffffffu, !ok);
    if (fail) acc = j0 + __ffs(fail) - 1;
  }
  int* emit = a.emit_tokens + (size_t)i * a.max_q_len;
  for (int j = lane; j < acc; j += 32) emit[j] = rm.row_next[q0 + j];
  if (lane == 0) {
    emit[acc] = key_col(a.row_best[q0 + acc]);
    a.accept_len[i] = acc;
    a.n_emit[i] = acc + 1;
  }
  for (int j = lane; j < n; j += 32) {
    const unsigned long long best = a.row_best[q0 + j];
    if (a.row_argmax) a.row_argmax[q0 + j] = key_col(best);
    if (a.row_zmax) a.row_zmax[q0 + j] = key_value(best);
    if (a.row_zdraft) a.row_zdraft[q0 + j] = a.zdraft[q0 + j];
  }
}
void launch_accept(cudaStream_t st, const AcceptArgs& a, const RowMeta& rm, const int* status, bool pdl) {
  launch_kernel(accept_kernel, dim3((a.n_seqs + 3) / 4), dim3(128), 0, st, pdl, a, rm, status);
}

// ------------------------------------------------------------------------------------------------
// Greedy traversal of a candidate tree (Eq. 9-12), one warp per sequence.  At the current node s: u_hat = the
// full-vocabulary argmax at s; u* = the child of s with the best score (exact mode: the child that carries u_hat);
// move to it iff z[u*] - z[u_hat] >= log tau; stop when the test fails or s has no child; emit pi(s) + u_hat.
__global__ void tree_accept_kernel(TreeAcceptArgs a, RowMeta rm, const int* status) {
  pdl_wait();               // everything below reads or writes what earlier kernels of the step produced
  pdl_launch_dependents();
  const int i = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (i >= a.n_seqs) return;
  const int lane = threadIdx.x & 31;
  if (*status) {            // a failed step decides nothing: the compaction and the commit that follow skip -1
    if (lane == 0) { a.accept_len[i] = -1; a.n_emit[i] = 0; }
    return;
  }
  const int q0 = rm.seq_q0[i], n = rm.seq_n[i], T = a.total_q;
  if (n <= 0) {
    if (lane == 0) { a.accept_len[i] = 0; a.n_emit[i] = 0; }
    return;
  }
  int* emit = a.emit_tokens + (size_t)i * a.max_q_len;
  int* path = a.accept_rows + (size_t)i * a.max_q_len;
  // every lane keeps four nodes (lane, lane + 32, ..) in registers: the walk itself then only fetches the row it
  // stands on
  constexpr int kPer = HSD_MAX_TREE_ROWS / 32;
  int npar[kPer], ntok[kPer];
  float nz[kPer];
#pragma unroll
  for (int k = 0; k < kPer; ++k) {
    const int c = lane + 32 * k;
    const bool in = c >= 1 && c < n;
    npar[k] = in ? a.parent[q0 + c] : -3;
    ntok[k] = in ? rm.row_tok[q0 + c] : -1;
    nz[k] = in ? a.zdraft[T + q0 + c] : 0.f;
  }
  int s = 0, acc = 0;
  for (int step = 0; step < n; ++step) {
    const unsigned long long best = a.row_best[q0 + s];
    const int uhat = key_col(best);
    int pick = -1, pick_tok = -1;
    float pick_z = 0.f;
    if (a.log_tau == 0.f) {
      // the child that carries u_hat (lowest row if a caller packed the same token twice under one parent)
      int mine = 0x7fffffff;
#pragma unroll
      for (int k = kPer - 1; k >= 0; --k)
        if (npar[k] == s && ntok[k] == uhat) mine = lane + 32 * k;
      for (int o = 16; o; o >>= 1) mine = min(mine, __shfl_xor_sync(0xffffffffu, mine, o));
      if (mine != 0x7fffffff) pick = mine;
    } else {
      // best child by (score, then lower token id), then lower row among equals
      unsigned long long bk = 0ull;
      int bc = 0x7fffffff;
#pragma unroll
      for (int k = 0; k < kPer; ++k) {
        if (npar[k] != s) continue;
        const unsigned long long key = argmax_key(nz[k], ntok[k]);
        if (bc == 0x7fffffff || key > bk) { bk = key; bc = lane + 32 * k; }
      }
      unsigned long long wk = bc != 0x7fffffff ? bk : 0ull;
      const unsigned has = __ballot_sync(0xffffffffu, bc != 0x7fffffff);
      for (int o = 16; o; o >>= 1) {
        const unsigned long long other = __shfl_xor_sync(0xffffffffu, wk, o);
        wk = other > wk ? other : wk;
      }
      if (has) {
        int lo = (bc != 0x7fffffff && bk == wk) ? bc : 0x7fffffff;
        for (int o = 16; o; o >>= 1) lo = min(lo, __shfl_xor_sync(0xffffffffu, lo, o));
        pick = lo;
      }
    }
    if (pick >= 0) {      // the owner lane broadcasts the node's token and score
      const int owner = pick & 31, k = pick >> 5;
      int tk = -1;
      float zk = 0.f;
#pragma unroll
      for (int kk = 0; kk < kPer; ++kk)
        if (kk == k) { tk = ntok[kk]; zk = nz[kk]; }
      pick_tok = __shfl_sync(0xffffffffu, tk, owner);
      pick_z = __shfl_sync(0xffffffffu, zk, owner);
      if (a.log_tau != 0.f && !(pick_z - key_value(best) >= a.log_tau)) pick = -1;
    }
    if (pick < 0) break;
    if (lane == 0) {
      path[acc] = pick;
      emit[acc] = pick_tok;
    }
    ++acc;
    s = pick;
  }
  if (lane == 0) {
    emit[acc] = key_col(a.row_best[q0 + s]);
    a.accept_len[i] = acc;
    a.n_emit[i] = acc + 1;
  }
  for (int j = lane; j < n; j += 32) {
    const unsigned long long best = a.row_best[q0 + j];
    if (a.row_argmax) a.row_argmax[q0 + j] = key_col(best);
    if (a.row_zmax) a.row_zmax[q0 + j] = key_value(best);
    if (a.row_zchild) a.row_zchild[q0 + j] = j > 0 ? a.zdraft[T + q0 + j] : __int_as_float(0x7fc00000);
  }
}
void launch_tree_accept(cudaStream_t st, const TreeAcceptArgs& a, const RowMeta& rm, const int* status, bool pdl) {
  launch_kernel(tree_accept_kernel, dim3((a.n_seqs + 3) / 4), dim3(128), 0, st, pdl, a, rm, status);
}

// KV maintenance after a tree step (Sec. 4.2: rollbacks and cache maintenance are part of the decode loop): the
// accepted path's rows move from their packed places L + r_d to the places L + d their rotary positions stand for.
// One CTA per (sequence, layer); a path's rows increase strictly, so moving depth by depth never overwrites a row
// that is still to be read.
__global__ void tree_compact_kernel(KvView kv, int n_kv_heads, int head_dim, int n_seqs, const int* seq_slots,
                                    const int* accept_len, const int* accept_rows, int max_q_len) {
  pdl_wait();               // everything below reads or writes what earlier kernels of the step produced
  pdl_launch_dependents();
  const int i = blockIdx.x, layer = blockIdx.y;
  const int slot = seq_slots ? seq_slots[i] : i;
  if (slot < 0 || slot >= kv.n_slots) return;
  const int a = accept_len[i];
  if (a < 0) return;                                     // the step failed a device-side check: nothing to keep
  const int L = kv.seq_lens[slot];
  if (L < 0 || (long long)L + max_q_len > (long long)kv.max_blocks * HSD_KV_BLOCK) return;
  const int* bt = kv.block_table + (size_t)slot * kv.max_blocks;
  const int row_chunks = head_dim / 8;                   // 16-byte chunks of one (token, kv head) row
  const int chunks = n_kv_heads * 2 * row_chunks;        // ... of one token's K and V rows in a layer
  for (int d = 1; d <= a && d < max_q_len; ++d) {
    const int r = accept_rows[(size_t)i * max_q_len + d - 1];
    if (r != d && r > 0 && r < max_q_len) {              // a row of this call (L + r is within the table, see above)
      const int ps = L + r, pd = L + d;
      const int bs = bt[ps / HSD_KV_BLOCK], bd = bt[pd / HSD_KV_BLOCK];
      if (bs >= 0 && bs < kv.n_blocks && bd >= 0 && bd < kv.n_blocks) {
        for (int t = threadIdx.x; t < chunks; t += blockDim.x) {
          const int c16 = t % row_chunks, pool = (t / row_chunks) & 1, h = t / (2 * row_chunks);
          bf16* base = pool ? kv.v_pool : kv.k_pool;
          const size_t src = ((((size_t)layer * kv.n_blocks + bs) * n_kv_heads + h) * 64 + ps % HSD_KV_BLOCK) * head_dim;
          const size_t dst = ((((size_t)layer * kv.n_blocks + bd) * n_kv_heads + h) * 64 + pd % HSD_KV_BLOCK) * head_dim;
          reinterpret_cast<uint4*>(base + dst)[c16] = reinterpret_cast<const uint4*>(base + src)[c16];
        }
      }
    }
    __syncthreads();
  }
}
void launch_tree_compact(cudaStream_t st, const KvView& kv, int n_layers, int n_kv_heads, int head_dim, int n_seqs,
                         const int* seq_slots, const int* accept_len, const int* accept_rows, int max_q_len, bool pdl) {
  launch_kernel(tree_compact_kernel, dim3(n_seqs, n_layers), dim3(128), 0, st, pdl, kv, n_kv_heads, head_dim, n_seqs, seq_slots,
                accept_len, accept_rows, max_q_len);
}

// ------------------------------------------------------------------------------------------------
// Draft-target matching and prefix-tree packing (Sec. 3.2, Eq. 5-7), one CTA per sequence.
//  1. the window takes in the tokens the last step emitted (w = the n most recent accepted tokens);
//  2. every position of the sequence's drafts where w occurs gives a candidate: the non-empty suffix after it
//     (Eq. 5, 6), in draft order then position order, at most kDsvMaxCands of them;
//  3. warp 0 grows the prefix tree level by level (Eq. 7): at depth d every live candidate moves to the child
//     that carries its d-th token, creating it while the node budget lasts; a candidate whose node cannot be
//     created stops.  Node ids are creation order, so parents precede children and the id is the packed row.
// Every sequence gets exactly max_rows rows: row 0 = the pending token, then the nodes, then padding rows
// (parent -2) that no traversal can enter.
constexpr int kDsvMaxCands = 64;
constexpr int kDsvMaxWindow = 8;
__global__ void dsv_build_kernel(DsvArgs a) {
  pdl_wait();               // everything below reads or writes what earlier kernels of the step produced
  pdl_launch_dependents();
  const int s = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  __shared__ int s_w[kDsvMaxWindow];
  __shared__ int s_cstart[kDsvMaxCands], s_clen[kDsvMaxCands], s_ccur[kDsvMaxCands];
  __shared__ int s_ntok[HSD_MAX_TREE_ROWS], s_npar[HSD_MAX_TREE_ROWS];
  __shared__ int s_ctok[kDsvMaxCands][HSD_MAX_TREE_ROWS];   // the part of every candidate a tree of this size can hold
  __shared__ unsigned s_ballot[4];
  __shared__ int s_ncand, s_nnodes;
  const int n = a.window_n;
  if (tid == 0) {
    // window <- last n of (window ++ emitted)
    int tmp[2 * kDsvMaxWindow];
    int m = 0;
    for (int i = 0; i < n; ++i) tmp[m++] = a.window[s * n + i];
    if (a.emit_tokens && a.n_emit) {
      const int ne = a.n_emit[s];
      for (int i = max(0, ne - n); i < ne; ++i) {
        if (m == 2 * kDsvMaxWindow) {
          for (int k = 1; k < m; ++k) tmp[k - 1] = tmp[k];
          --m;
        }
        tmp[m++] = a.emit_tokens[(size_t)s * a.emit_stride + i];
      }
    }
    for (int i = 0; i < n; ++i) {
      s_w[i] = tmp[m - n + i];
      a.window[s * n + i] = s_w[i];
    }
    s_ncand = 0;
    s_nnodes = 0;
    a.cu_q[s] = s * a.max_rows;
    if (s == 0) a.cu_q[a.n_seqs] = a.n_seqs * a.max_rows;
  }
  __syncthreads();
  bool have_w = true;
  for (int i = 0; i < n; ++i) have_w = have_w && s_w[i] >= 0;
  // ---- candidates
  if (have_w) {
    // every offset is clamped to the array sizes the host passed: a malformed table shortens or drops drafts
    // whose drafts: the sequence's own, or (lane batches) those of the owner the map names; -1 or out of range = none
    const int owner = a.seq_map ? a.seq_map[s] : s;
    const bool owned = a.seq_map ? (owner >= 0 && owner < a.n_owners) : true;
    const int d_lo = owned ? min(max(a.seq_draft_off[owner], 0), a.n_drafts) : 0;
    const int d_hi = owned ? min(max(a.seq_draft_off[owner + 1], 0), a.n_drafts) : 0;
    for (int d = d_lo; d < d_hi; ++d) {
      const int d0 = min(max(a.draft_off[d], 0), a.total_draft_tokens);
      const int len = min(max(a.draft_off[d + 1], d0), a.total_draft_tokens) - d0;
      for (int j0 = 0; j0 + n < len; j0 += blockDim.x) {      // j + n < len: a non-empty suffix follows the window
        if (s_ncand >= kDsvMaxCands) break;
        const int j = j0 + tid;
        bool hit = j + n < len;
        for (int i = 0; hit && i < n; ++i) hit = a.draft_tokens[d0 + j + i] == s_w[i];
        const unsigned b = __ballot_sync(0xffffffffu, hit);
        if (lane == 0) s_ballot[warp] = b;
        __syncthreads();
        int before = s_ncand;
        for (int w = 0; w < warp; ++w) before += __popc(s_ballot[w]);
        const int slot = before + __popc(b & ((1u << lane) - 1u));
        if (hit && slot < kDsvMaxCands) {
          s_cstart[slot] = d0 + j + n;
          s_clen[slot] = len - (j + n);
          s_ccur[slot] = 0;
        }
        __syncthreads();
        if (tid == 0) {
          int tot = s_ncand;
          for (int w = 0; w < (int)(blockDim.x >> 5); ++w) tot += __popc(s_ballot[w]);
          s_ncand = min(tot, kDsvMaxCands);
        }
        __syncthreads();
      }
    }
  }
  __syncthreads();
  for (int idx = tid; idx < s_ncand * HSD_MAX_TREE_ROWS; idx += blockDim.x) {
    const int c = idx / HSD_MAX_TREE_ROWS, d = idx % HSD_MAX_TREE_ROWS;
    s_ctok[c][d] = d < s_clen[c] ? a.draft_tokens[s_cstart[c] + d] : -1;
  }
  __syncthreads();
  // ---- prefix tree, level by level (warp 0; node ids 1.. in creation order, id 0 = root)
  if (warp == 0) {
    const int ncand = s_ncand, budget = a.max_rows - 1;
    int nn = 0;
    unsigned long long alive = ncand >= 64 ? ~0ull : ((1ull << ncand) - 1ull);
    for (int depth = 0; alive && depth < HSD_MAX_TREE_ROWS; ++depth) {
      const int level0 = nn + 1;       // a node's children are all created while its level is expanded: search only those
      for (int c = 0; c < ncand; ++c) {
        if (!((alive >> c) & 1ull)) continue;
        if (depth >= s_clen[c]) { alive &= ~(1ull << c); continue; }
        const int u = s_ctok[c][depth];
        const int cur = s_ccur[c];
        int found = 0;
        for (int base = level0; base <= nn && !found; base += 32) {
          const int id = base + lane;
          const bool hit = id <= nn && s_npar[id] == cur && s_ntok[id] == u;
          const unsigned m = __ballot_sync(0xffffffffu, hit);
          if (m) found = base + __ffs(m) - 1;
        }
        if (!found) {
          if (nn >= budget) { alive &= ~(1ull << c); continue; }
          ++nn;
          if (lane == 0) { s_ntok[nn] = u; s_npar[nn] = cur; }
          found = nn;
        }
        if (lane == 0) s_ccur[c] = found;
        __syncwarp();
      }
    }
    if (lane == 0) s_nnodes = nn;
  }
  __syncthreads();
  // ---- packed rows
  const int nn = s_nnodes, pending = s_w[n - 1];
  for (int r = tid; r < a.max_rows; r += blockDim.x) {
    const size_t o = (size_t)s * a.max_rows + r;
    if (r == 0) { a.q_tokens[o] = pending; a.parent[o] = -1; }
    else if (r <= nn) { a.q_tokens[o] = s_ntok[r]; a.parent[o] = s_npar[r]; }
    else { a.q_tokens[o] = pending; a.parent[o] = -2; }
  }
  if (tid == 0) a.n_rows[s] = nn + 1;
}
void launch_dsv_build(cudaStream_t st, const DsvArgs& a, bool pdl) {
  launch_kernel(dsv_build_kernel, dim3(a.n_seqs), dim3(128), 0, st, pdl, a);
}

// ------------------------------------------------------------------------------------------------
// Lane batches (Sec. 3.1, Stage 1: many regions, each decoded to its end by repeated steps).  A lane serves one
// sequence at a time; between two steps one CTA appends what every lane's sequence emitted, counts the step, retires
// the sequences that have reached their length and hands free lanes to waiting sequences in queue order.
// counters: [0] next waiting sequence, [1] sequences not finished, [2] steps taken.
__device__ void stage_assign_lanes(const StageDev& sd, const KvView& kv) {      // one thread, lanes in order
  int head = sd.counters[0], left = sd.counters[1];
  for (int i = 0; i < sd.n_lanes; ++i) {
    const int r = sd.lane_seq[i];
    if (r >= 0 && sd.out_len[r] < sd.max_new[r]) continue;                      // still decoding
    if (r >= 0) --left;                                                         // finished in this step
    int nxt = -1;
    while (head < sd.n_seqs && nxt < 0) {
      if (sd.out_len[head] < sd.max_new[head]) nxt = head; else --left;         // (a sequence of length <= 1 is done at once)
      ++head;
    }
    sd.lane_seq[i] = nxt;
    const int slot = nxt < 0 ? sd.idle_slot : (sd.seq_slot ? sd.seq_slot[nxt] : nxt);
    sd.lane_slot[i] = slot;
    for (int k = 0; k < sd.window_n; ++k) sd.window[i * sd.window_n + k] = -1;
    sd.window[i * sd.window_n + sd.window_n - 1] = nxt < 0 ? 0 : sd.first_token[nxt];
  }
  sd.counters[0] = head;
  sd.counters[1] = left;
  if (sd.idle_slot >= 0 && sd.idle_slot < kv.n_slots) kv.seq_lens[sd.idle_slot] = 0;   // idle lanes restart from an empty cache
}

__global__ void stage_begin_kernel(StageDev sd, KvView kv) {
  pdl_wait();               // everything below reads or writes what earlier kernels of the step produced
  pdl_launch_dependents();
  for (int r = threadIdx.x; r < sd.n_seqs; r += blockDim.x) {
    sd.out_tokens[(size_t)r * sd.out_stride] = sd.first_token[r];
    sd.out_len[r] = 1;
    sd.seq_steps[r] = 0;
    sd.seq_accepted[r] = 0;
  }
  for (int i = threadIdx.x; i < sd.n_lanes; i += blockDim.x) sd.lane_seq[i] = -1;
  if (threadIdx.x == 0) {
    sd.counters[0] = 0;
    sd.counters[1] = sd.n_seqs;
    sd.counters[2] = 0;
  }
  __syncthreads();
  if (threadIdx.x == 0) stage_assign_lanes(sd, kv);
}
void launch_stage_begin(cudaStream_t st, const StageDev& sd, const KvView& kv, bool pdl) {
  launch_kernel(stage_begin_kernel, dim3(1), dim3(128), 0, st, pdl, sd, kv);
}

__global__ void stage_advance_kernel(StageDev sd, KvView kv, const int* accept_len, const int* emit_tokens,
                                     const int* n_emit, int emit_stride) {
  pdl_wait();               // everything below reads or writes what earlier kernels of the step produced
  pdl_launch_dependents();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, n_warps = blockDim.x >> 5;
  for (int i = warp; i < sd.n_lanes; i += n_warps) {       // one warp per lane
    const int r = sd.lane_seq[i];
    if (r < 0 || r >= sd.n_seqs) continue;
    const int a = accept_len[i];
    if (a < 0) continue;                                   // the step failed a device-side check: nothing was decided
    const int have = sd.out_len[r];
    const int room = max(0, min(sd.max_new[r], sd.out_stride) - have);
    const int take = min(max(n_emit[i], 0), room);
    for (int k = lane; k < take; k += 32) sd.out_tokens[(size_t)r * sd.out_stride + have + k] = emit_tokens[(size_t)i * emit_stride + k];
    __syncwarp();
    if (lane == 0) {
      sd.out_len[r] = have + take;
      sd.seq_steps[r] += 1;
      sd.seq_accepted[r] += min(a, room);
      // the window keeps the most recent accepted tokens, the pending one last
      const int n = sd.window_n;
      for (int k = 0; k < n; ++k) {
        const int back = n - 1 - k;                        // token `back` places before the newest
        const int idx = have + take - 1 - back;
        sd.window[i * n + k] = idx >= 0 ? sd.out_tokens[(size_t)r * sd.out_stride + idx] : -1;
      }
    }
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    sd.counters[2] += 1;
    stage_assign_lanes(sd, kv);
  }
}
void launch_stage_advance(cudaStream_t st, const StageDev& sd, const KvView& kv, const int* accept_len,
                          const int* emit_tokens, const int* n_emit, int emit_stride, bool pdl) {
  launch_kernel(stage_advance_kernel, dim3(1), dim3(256), 0, st, pdl, sd, kv, accept_len, emit_tokens, n_emit, emit_stride);
}

// The page draft of Stage 2 (Eq. 3): the outputs of all sequences, concatenated, with their offsets.
__global__ void stage_aggregate_kernel(StageDev sd, int* draft_tokens, int capacity, int* draft_off) {
  pdl_wait();               // everything below reads or writes what earlier kernels of the step produced
  pdl_launch_dependents();
  __shared__ int s_off;
  if (threadIdx.x == 0) {
    int off = 0;
    for (int r = 0; r < sd.n_seqs; ++r) {                  // serial scan: a page has tens of regions
      draft_off[r] = off;
      off = min(capacity, off + max(0, min(sd.out_len[r], sd.out_stride)));
    }
    draft_off[sd.n_seqs] = off;
    s_off = off;
  }
  __syncthreads();
  for (int r = 0; r < sd.n_seqs; ++r) {
    const int lo = draft_off[r], n = draft_off[r + 1] - lo;
    for (int k = threadIdx.x; k < n; k += blockDim.x) draft_tokens[lo + k] = sd.out_tokens[(size_t)r * sd.out_stride + k];
  }
}
void launch_stage_aggregate(cudaStream_t st, const StageDev& sd, int* draft_tokens, int capacity, int* draft_off, bool pdl) {
  launch_kernel(stage_aggregate_kernel, dim3(1), dim3(256), 0, st, pdl, sd, draft_tokens, capacity, draft_off);
}

// Prefill epilogue: first pending token per sequence, and seq_lens += rows.
__global__ void first_token_kernel(const unsigned long long* row_best, int n_seqs, int* first_token, RowMeta rm,
                                   KvView kv, const int* status) {
  pdl_wait();               // everything below reads or writes what earlier kernels of the step produced
  pdl_launch_dependents();
  if (*status) return;
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n_seqs) return;
  first_token[i] = key_col(row_best[i]);
  kv.seq_lens[rm.seq_slot[i]] = rm.seq_len[i] + rm.seq_n[i];
}
void launch_first_token(cudaStream_t st, const unsigned long long* row_best, int n_seqs, int* first_token,
                        const RowMeta& rm, const KvView& kv, const int* status, bool pdl) {
  launch_kernel(first_token_kernel, dim3((n_seqs + 127) / 128), dim3(128), 0, st, pdl, row_best, n_seqs, first_token, rm,
                kv, status);
}

// ------------------------------------------------------------------------------------------------
// KV commit / rollback: the pending row and the accepted rows stay, the rest is dead and gets overwritten.
__global__ void commit_kernel(KvView kv, int n_seqs, const int* seq_slots, const int* accept_len, int* blocks_in_use) {
  pdl_wait();               // everything below reads or writes what earlier kernels of the step produced
  pdl_launch_dependents();
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n_seqs) return;
  const int slot = seq_slots ? seq_slots[i] : i;
  if (slot < 0 || slot >= kv.n_slots) return;
  const int a = accept_len[i];
  int L = kv.seq_lens[slot];
  if (a >= 0) L = min(L + a + 1, kv.max_blocks * HSD_KV_BLOCK);
  kv.seq_lens[slot] = L;
  if (blocks_in_use) blocks_in_use[i] = (L + HSD_KV_BLOCK - 1) / HSD_KV_BLOCK;
}
void launch_commit(cudaStream_t st, const KvView& kv, int n_seqs, const int* seq_slots, const int* accept_len,
                   int* blocks_in_use, bool pdl) {
  launch_kernel(commit_kernel, dim3((n_seqs + 127) / 128), dim3(128), 0, st, pdl, kv, n_seqs, seq_slots, accept_len,
                blocks_in_use);
}

}  // namespace hsd
