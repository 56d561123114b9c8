// Kernels of the adaptive-LayerNorm transformer (DiT-style action expert) that the decoder-style
// network does not have: modulated LayerNorm, the modulated output head, cross-attention to a long
// context (up to 256 tokens), SiLU.  The timestep enters only through tables built at weight load:
// mod [T, L*6d + 2d] holds, for every timestep, each block's (shift1, scale1, gate1, shift2, scale2,
// gate2) and the final layer's (shift, scale).
#pragma once
#include "common.cuh"
#include "net_kernels.cuh"

namespace tsdp {

__global__ void silu_inplace_kernel(float* __restrict__ x, long long n) {
  pdl_trigger();
  pdl_wait();
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) x[i] = x[i] / (1.0f + expf(-x[i]));
}

__device__ __forceinline__ int row_tau(const CandMap& cm, int row, int H, int Tsteps) {
  int b, c;
  cand_decode(cm, row / H, b, c);
  const int tau = cm.t[b] - cm.koff - c;
  return max(0, min(Tsteps - 1, tau));
}

// out[row] = LN0(h[row]) * (1 + scale(tau)) + shift(tau); LN0 = LayerNorm without gain and bias.
// One warp per row, d = VEC * 128; shift / scale are columns [off_shift, +d) and [off_scale, +d) of mod[tau].
template <typename T, int VEC>
__global__ void ln_mod_kernel(const float* __restrict__ h, const float* __restrict__ mod, int mod_ld, int off_shift,
                              int off_scale, CandMap cm, int H, int Tsteps, T* __restrict__ out, int M) {
  pdl_trigger();
  pdl_wait();
  constexpr int d = VEC * 128;
  const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (row >= M || row / H >= cand_count(cm, M / H)) return;
  float4 v[VEC];
  float s = 0.f;
#pragma unroll
  for (int j = 0; j < VEC; ++j) {
    v[j] = reinterpret_cast<const float4*>(h + (size_t)row * d)[j * 32 + lane];
    s += v[j].x + v[j].y + v[j].z + v[j].w;
  }
  const float mean = warp_sum(s) / d;
  float q = 0.f;
#pragma unroll
  for (int j = 0; j < VEC; ++j) {
    v[j].x -= mean; v[j].y -= mean; v[j].z -= mean; v[j].w -= mean;
    q += v[j].x * v[j].x + v[j].y * v[j].y + v[j].z * v[j].z + v[j].w * v[j].w;
  }
  const float rstd = rsqrtf(warp_sum(q) / d + 1e-5f);
  const float* mrow = mod + (size_t)row_tau(cm, row, H, Tsteps) * mod_ld;
#pragma unroll
  for (int j = 0; j < VEC; ++j) {
    const int c = (j * 32 + lane) * 4;
    const float4 sh = __ldg(reinterpret_cast<const float4*>(mrow + off_shift + c));
    const float4 sc = __ldg(reinterpret_cast<const float4*>(mrow + off_scale + c));
    store4(out + (size_t)row * d + c, v[j].x * rstd * (1.0f + sc.x) + sh.x, v[j].y * rstd * (1.0f + sc.y) + sh.y,
           v[j].z * rstd * (1.0f + sc.z) + sh.z, v[j].w * rstd * (1.0f + sc.w) + sh.w);
  }
}

// eps[n, i, :] = (LN0(h[row]) (1 + scale_f(tau)) + shift_f(tau)) W_out + b_out; one warp per row.
template <int VEC>
__global__ void head_mod_kernel(const float* __restrict__ h, const float* __restrict__ mod, int mod_ld, int off_shift,
                                int off_scale, const float* __restrict__ W_outT, const float* __restrict__ b_out,
                                CandMap cm, int M, int H, int A, int Tsteps) {
  pdl_trigger();
  pdl_wait();
  constexpr int d = VEC * 128;
  const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (row >= M || row / H >= cand_count(cm, M / H)) return;
  float4 v[VEC];
  float s = 0.f;
#pragma unroll
  for (int j = 0; j < VEC; ++j) {
    v[j] = reinterpret_cast<const float4*>(h + (size_t)row * d)[j * 32 + lane];
    s += v[j].x + v[j].y + v[j].z + v[j].w;
  }
  const float mean = warp_sum(s) / d;
  float q = 0.f;
#pragma unroll
  for (int j = 0; j < VEC; ++j) {
    v[j].x -= mean; v[j].y -= mean; v[j].z -= mean; v[j].w -= mean;
    q += v[j].x * v[j].x + v[j].y * v[j].y + v[j].z * v[j].z + v[j].w * v[j].w;
  }
  const float rstd = rsqrtf(warp_sum(q) / d + 1e-5f);
  const float* mrow = mod + (size_t)row_tau(cm, row, H, Tsteps) * mod_ld;
#pragma unroll
  for (int j = 0; j < VEC; ++j) {
    const int c = (j * 32 + lane) * 4;
    const float4 sh = __ldg(reinterpret_cast<const float4*>(mrow + off_shift + c));
    const float4 sc = __ldg(reinterpret_cast<const float4*>(mrow + off_scale + c));
    v[j].x = v[j].x * rstd * (1.0f + sc.x) + sh.x; v[j].y = v[j].y * rstd * (1.0f + sc.y) + sh.y;
    v[j].z = v[j].z * rstd * (1.0f + sc.z) + sh.z; v[j].w = v[j].w * rstd * (1.0f + sc.w) + sh.w;
  }
  const int n = row / H, i = row % H;
  int b, c;
  cand_decode(cm, n, b, c);
  float* o = cm.eout + b * cm.e_stride_b + (long long)c * H * A + (long long)i * A;
  for (int a = 0; a < A; ++a) {
    float acc = 0.f;
#pragma unroll
    for (int j = 0; j < VEC; ++j) {
      const float4 w = reinterpret_cast<const float4*>(W_outT + (size_t)a * d)[j * 32 + lane];
      acc += v[j].x * w.x + v[j].y * w.y + v[j].z * w.z + v[j].w * w.w;
    }
    acc = warp_sum(acc);
    if (lane == 0) o[a] = acc + b_out[a];
  }
}

// ------------------------------------------------------------------------------------------------
// Cross-attention to the context tokens of a request, any type (check mode and odd head widths): one
// warp per query row and head, keys strided over the lanes, two passes (scores, then values).
// q, out [M, d]; kv [items * Tc, ld_kv] with this block's [K (d) | V (d)] at column kv_off.
// ------------------------------------------------------------------------------------------------
template <typename T>
__global__ void cross_attn_ctx_simt_kernel(const T* __restrict__ q, T* __restrict__ out, const T* __restrict__ kv,
                                           long long ld_kv, int kv_off, CandMap cm, int M, int H, int d, int heads, int Tc) {
  pdl_trigger();
  pdl_wait();
  extern __shared__ float sm_ctx[];                       // per warp: Tc scores
  const int wpb = blockDim.x >> 5, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int row = blockIdx.x * wpb + warp;
  if (row >= M || row / H >= cand_count(cm, M / H)) return;
  int b, c_unused;
  cand_decode(cm, row / H, b, c_unused);
  const int dh = d / heads;
  const T* kvb = kv + (size_t)item_of(cm.item, b) * Tc * ld_kv + kv_off;
  float* sc = sm_ctx + (size_t)warp * Tc;
  const float scale = rsqrtf((float)dh);
  for (int hd = 0; hd < heads; ++hd) {
    const T* qp = q + (size_t)row * d + hd * dh;
    float m = -INFINITY;
    for (int k = lane; k < Tc; k += 32) {
      const T* kp = kvb + (size_t)k * ld_kv + hd * dh;
      float a = 0.f;
      for (int i = 0; i < dh; ++i) a += to_f(qp[i]) * to_f(kp[i]);
      sc[k] = a * scale;
      m = fmaxf(m, sc[k]);
    }
    m = warp_max(m);
    float l = 0.f;
    for (int k = lane; k < Tc; k += 32) { sc[k] = __expf(sc[k] - m); l += sc[k]; }
    l = warp_sum(l);
    __syncwarp();
    const float inv = 1.0f / l;
    for (int i = lane; i < dh; i += 32) {
      float o = 0.f;
      for (int k = 0; k < Tc; ++k) o += sc[k] * to_f(kvb[(size_t)k * ld_kv + d + hd * dh + i]);
      out[(size_t)row * d + hd * dh + i] = from_f<T>(o * inv);
    }
    __syncwarp();
  }
}

// ------------------------------------------------------------------------------------------------
// Tensor-core cross-attention to the context (bf16): one block per (slot, head) keeps that head's keys
// and values of the slot's request in shared memory; each warp takes 16-query tiles of the slot's
// C * H query rows and runs S = Q K^T and O = P V on mma.sync over 64-key chunks with an online
// softmax.  Tc <= 256, a multiple of 16.
// ------------------------------------------------------------------------------------------------
constexpr int CX_WARPS = 8;
template <int DH>
__host__ __device__ constexpr int cx_smem_bytes(int Tc) { return 2 * Tc * (DH + 8) * 2; }

template <int DH>
__global__ void __launch_bounds__(CX_WARPS * 32)
cross_attn_ctx_mma_kernel(const __nv_bfloat16* __restrict__ q, __nv_bfloat16* __restrict__ out,
                          const __nv_bfloat16* __restrict__ kv, long long ld_kv, int kv_off, CandMap cm, int rows_per_slot,
                          int d, int heads, int Tc, const int* __restrict__ slot_start, int H) {
  pdl_trigger();
  pdl_wait();
  extern __shared__ __align__(16) uint8_t cx_raw[];
  constexpr int P = DH + 8, KS = DH / 16, NO = DH / 8;
  constexpr int CX_U = 1;      // query tiles a warp processes together (2 costs more in occupancy than it saves in shared-memory reads)
  __nv_bfloat16* Ks = reinterpret_cast<__nv_bfloat16*>(cx_raw);
  __nv_bfloat16* Vs = Ks + (size_t)Tc * P;
  int b = blockIdx.x / heads;
  const int hd = blockIdx.x % heads;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, tg = lane & 3;
  // Rows of group b.  Dense layout: slot b owns [b * rows_per_slot, +rows_per_slot).  Compacted candidate list
  // with slot_start: slot b's candidates are the list entries slot_start[b] .. slot_start[b + 1] - 1, H rows each.
  // Compacted list without slot_start (one candidate per slot, C = 1): group b is list entry b, slot list[b] >> 6.
  size_t row0 = (size_t)b * rows_per_slot;
  if (slot_start != nullptr) {
    row0 = (size_t)slot_start[b] * H;
    rows_per_slot = (slot_start[b + 1] - slot_start[b]) * H;
    if (rows_per_slot <= 0) return;
  } else if (cm.list != nullptr) {
    if (b >= cand_count(cm, (int)(gridDim.x / heads))) return;
    b = cm.list[b] >> 6;
  }
  const __nv_bfloat16* kvb = kv + (size_t)item_of(cm.item, b) * Tc * ld_kv + kv_off + hd * DH;
  constexpr int VPR = DH / 8;
  for (int i = threadIdx.x; i < Tc * VPR; i += blockDim.x) {
    const int r = i / VPR, v = i % VPR;
    *reinterpret_cast<uint4*>(Ks + (size_t)r * P + v * 8) = __ldg(reinterpret_cast<const uint4*>(kvb + (size_t)r * ld_kv) + v);
    *reinterpret_cast<uint4*>(Vs + (size_t)r * P + v * 8) = __ldg(reinterpret_cast<const uint4*>(kvb + (size_t)r * ld_kv + d) + v);
  }
  __syncthreads();
  const float scale = rsqrtf((float)DH);
  // A warp works on CX_U query tiles at a time, so that every key / value fragment read from shared
  // memory feeds CX_U tensor-core instructions.
  for (int pt = warp; pt * (16 * CX_U) < rows_per_slot; pt += CX_WARPS) {
    int r0[CX_U], r1[CX_U];
    bool v0[CX_U], v1[CX_U];
    uint32_t qa[CX_U][KS][4];
    float o[CX_U][NO][4];
    float m0[CX_U], m1[CX_U], l0[CX_U], l1[CX_U];
#pragma unroll
    for (int u = 0; u < CX_U; ++u) {
      r0[u] = (pt * CX_U + u) * 16 + g; r1[u] = r0[u] + 8;
      v0[u] = r0[u] < rows_per_slot; v1[u] = r1[u] < rows_per_slot;
      const __nv_bfloat16* q0 = q + (row0 + r0[u]) * d + hd * DH;
      const __nv_bfloat16* q1 = q + (row0 + r1[u]) * d + hd * DH;
#pragma unroll
      for (int ks = 0; ks < KS; ++ks) {
        const int c = ks * 16 + 2 * tg;
        qa[u][ks][0] = v0[u] ? *reinterpret_cast<const uint32_t*>(q0 + c) : 0u;
        qa[u][ks][1] = v1[u] ? *reinterpret_cast<const uint32_t*>(q1 + c) : 0u;
        qa[u][ks][2] = v0[u] ? *reinterpret_cast<const uint32_t*>(q0 + c + 8) : 0u;
        qa[u][ks][3] = v1[u] ? *reinterpret_cast<const uint32_t*>(q1 + c + 8) : 0u;
      }
#pragma unroll
      for (int no = 0; no < NO; ++no) o[u][no][0] = o[u][no][1] = o[u][no][2] = o[u][no][3] = 0.f;
      m0[u] = m1[u] = -INFINITY; l0[u] = l1[u] = 0.f;
    }
    for (int k0 = 0; k0 < Tc; k0 += 64) {
      float s[CX_U][8][4];
#pragma unroll
      for (int nt = 0; nt < 8; ++nt) {
#pragma unroll
        for (int u = 0; u < CX_U; ++u) s[u][nt][0] = s[u][nt][1] = s[u][nt][2] = s[u][nt][3] = 0.f;
        if (k0 + nt * 8 < Tc) {
#pragma unroll
          for (int ks = 0; ks < KS; ks += 2) {
            uint32_t bk[4];
            ldmatrix_x4(bk, Ks + (size_t)(k0 + nt * 8 + (lane & 7)) * P + ks * 16 + 8 * (lane >> 3));
#pragma unroll
            for (int u = 0; u < CX_U; ++u) {
              mma_bf16_16816(s[u][nt], qa[u][ks], bk[0], bk[1]);
              mma_bf16_16816(s[u][nt], qa[u][ks + 1], bk[2], bk[3]);
            }
          }
        }
      }
#pragma unroll
      for (int u = 0; u < CX_U; ++u) {
        float cm0 = -INFINITY, cm1 = -INFINITY;
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
          const bool vis = k0 + nt * 8 < Tc;                  // Tc is a multiple of 16: a tile is all in or all out
#pragma unroll
          for (int e = 0; e < 4; ++e) s[u][nt][e] = vis ? s[u][nt][e] * scale : -INFINITY;
          cm0 = fmaxf(cm0, fmaxf(s[u][nt][0], s[u][nt][1]));
          cm1 = fmaxf(cm1, fmaxf(s[u][nt][2], s[u][nt][3]));
        }
        cm0 = fmaxf(cm0, __shfl_xor_sync(0xffffffffu, cm0, 1)); cm0 = fmaxf(cm0, __shfl_xor_sync(0xffffffffu, cm0, 2));
        cm1 = fmaxf(cm1, __shfl_xor_sync(0xffffffffu, cm1, 1)); cm1 = fmaxf(cm1, __shfl_xor_sync(0xffffffffu, cm1, 2));
        const float n0 = fmaxf(m0[u], cm0), n1 = fmaxf(m1[u], cm1);
        const float f0 = __expf(m0[u] - n0), f1 = __expf(m1[u] - n1);   // exp(-inf) = 0 on the first chunk
        m0[u] = n0; m1[u] = n1;
        float a0 = 0.f, a1 = 0.f;
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
          s[u][nt][0] = __expf(s[u][nt][0] - n0); s[u][nt][1] = __expf(s[u][nt][1] - n0);
          s[u][nt][2] = __expf(s[u][nt][2] - n1); s[u][nt][3] = __expf(s[u][nt][3] - n1);
          a0 += s[u][nt][0] + s[u][nt][1]; a1 += s[u][nt][2] + s[u][nt][3];
        }
        a0 += __shfl_xor_sync(0xffffffffu, a0, 1); a0 += __shfl_xor_sync(0xffffffffu, a0, 2);
        a1 += __shfl_xor_sync(0xffffffffu, a1, 1); a1 += __shfl_xor_sync(0xffffffffu, a1, 2);
        l0[u] = l0[u] * f0 + a0; l1[u] = l1[u] * f1 + a1;
#pragma unroll
        for (int no = 0; no < NO; ++no) { o[u][no][0] *= f0; o[u][no][1] *= f0; o[u][no][2] *= f1; o[u][no][3] *= f1; }
      }
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        if (k0 + 16 * j < Tc) {
          uint32_t pa[CX_U][4];
#pragma unroll
          for (int u = 0; u < CX_U; ++u) {
            pa[u][0] = pack_bf16(s[u][2 * j][0], s[u][2 * j][1]); pa[u][1] = pack_bf16(s[u][2 * j][2], s[u][2 * j][3]);
            pa[u][2] = pack_bf16(s[u][2 * j + 1][0], s[u][2 * j + 1][1]); pa[u][3] = pack_bf16(s[u][2 * j + 1][2], s[u][2 * j + 1][3]);
          }
#pragma unroll
          for (int no = 0; no < NO; no += 2) {
            uint32_t bv[4];
            ldmatrix_x4_trans(bv, Vs + (size_t)(k0 + 16 * j + (lane & 7) + 8 * ((lane >> 3) & 1)) * P + no * 8 + 8 * (lane >> 4));
#pragma unroll
            for (int u = 0; u < CX_U; ++u) {
              mma_bf16_16816(o[u][no], pa[u], bv[0], bv[1]);
              mma_bf16_16816(o[u][no + 1], pa[u], bv[2], bv[3]);
            }
          }
        }
      }
    }
#pragma unroll
    for (int u = 0; u < CX_U; ++u) {
      const float i0 = 1.0f / l0[u], i1 = 1.0f / l1[u];
      __nv_bfloat16* o0 = out + (row0 + r0[u]) * d + hd * DH;
      __nv_bfloat16* o1 = out + (row0 + r1[u]) * d + hd * DH;
#pragma unroll
      for (int no = 0; no < NO; ++no) {
        const int col = no * 8 + 2 * tg;
        if (v0[u]) *reinterpret_cast<uint32_t*>(o0 + col) = pack_bf16(o[u][no][0] * i0, o[u][no][1] * i0);
        if (v1[u]) *reinterpret_cast<uint32_t*>(o1 + col) = pack_bf16(o[u][no][2] * i1, o[u][no][3] * i1);
      }
    }
  }
}

}  // namespace tsdp
