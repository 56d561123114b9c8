// Cross-attention sub-block of the decoder transformer with the projections folded into the memory
// tokens.  The block is
//     x <- x + softmax_j( q_h . k_{j,h} / sqrt(dh) ) v_{j,h}  Wo2 + bo2,      q = LN2(x) Wq2 + bq2,
// with only NK = 1 + obs_tokens memory tokens j (the time token and the observation tokens), whose
// keys k_j and values v_j do not depend on x.  Because NK is tiny, both d x d projections can be
// applied to the memory tokens instead of to every token row:
//     score_{h,j}(x) = xhat . kq_{j,h} + c_{j,h},      xhat = (x - mean) rstd   (LayerNorm without its affine part)
//         kq_{j,h}[i] = g2[i] * sum_{c in head h} Wq2[i, c] k_j[c] / sqrt(dh)
//         c_{j,h}     = sum_{c in head h} (bq2[c] + sum_i b2[i] Wq2[i, c]) k_j[c] / sqrt(dh)
//     out(x) = sum_{h,j} p_{h,j} u_{j,h} + bo2,         u_{j,h}[o] = sum_{c in head h} v_j[c] Wo2[c, o]
// so the LayerNorm, the query GEMM, the attention and the output GEMM become one pass over the
// residual stream: two small tensor-core products per candidate, [16 x d] x [d x NK*heads] and
// [16 x NK*heads] x [NK*heads x d].  The vectors kq, u and the constants c are tabulated per memory
// token and block: for every timestep when the weights are loaded (time token), for every request
// when its observation arrives (observation tokens).
//
// Table layouts (bf16 unless noted), `row` = timestep or request * obs_tokens + token:
//   kq [row][layer][heads][d]           a lane's B fragments of consecutive k steps are 32 bytes apart
//   ut [row][layer][heads/2][d][2]      u transposed, heads in pairs: a lane's B fragments of consecutive 8-column
//                                       tiles are 32 bytes apart, and 8 lanes read one full 32-byte sector
//   cc [row][layer][heads]  fp32
#pragma once
#include "common.cuh"
#include "net_kernels.cuh"

namespace tsdp {

constexpr int XF_THREADS = 128;
constexpr int XF_MAXN = 32;          // (1 + obs_tokens) * heads at most
constexpr int XF_MAXNK = 4;          // 1 + obs_tokens at most
constexpr int XF_RB = 4;             // memory tokens per pass of the table builder

struct XfoldLayerW {
  const __nv_bfloat16* Wq2;          // [d out][d in]
  const __nv_bfloat16* Wo2;          // [d out][d in]
  const float* bq2;
  const float* ln_g;
  const float* ln_b;
};

struct XfoldTables {
  const __nv_bfloat16 *kq_time, *ut_time;
  const float* c_time;
  const __nv_bfloat16 *kq_obs, *ut_obs;
  const float* c_obs;
};

__host__ __device__ constexpr size_t xfold_build_smem(int d, int dh) { return (size_t)2 * dh * d * 2 + (size_t)(2 * XF_RB + 1) * dh * 4; }

// Tables of `rows` memory tokens whose keys / values are kv[row][layer][k (d) | v (d)] (fp32, row pitch ldkv).
// grid (layers * heads, row splits), 256 threads; a block keeps its head's slice of Wq2 and Wo2 in shared memory.
__global__ void __launch_bounds__(256)
xfold_build_kernel(const float* __restrict__ kv, long long ldkv, int rows, const XfoldLayerW* __restrict__ lw, int L, int d,
                   int heads, __nv_bfloat16* __restrict__ kq, __nv_bfloat16* __restrict__ ut, float* __restrict__ cc) {
  extern __shared__ __align__(16) unsigned char xf_smem[];
  const int DH = d / heads;
  const int layer = blockIdx.x / heads, h = blockIdx.x % heads;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  __nv_bfloat16* sWq = reinterpret_cast<__nv_bfloat16*>(xf_smem);   // [DH][d]: sWq[c][i] = Wq2[in i, out h DH + c]
  __nv_bfloat16* sWo = sWq + (size_t)DH * d;                        // [DH][d]: sWo[c][o] = Wo2[in h DH + c, out o]
  float* sk = reinterpret_cast<float*>(sWo + (size_t)DH * d);       // [k | v][DH][XF_RB memory tokens]
  float* swb = sk + 2 * DH * XF_RB;                                         // bq2 + b2 . Wq2, this head [DH]
  const XfoldLayerW w = lw[layer];
  {
    const uint4* src = reinterpret_cast<const uint4*>(w.Wq2 + (size_t)h * DH * d);
    for (int idx = threadIdx.x; idx < DH * d / 8; idx += blockDim.x) reinterpret_cast<uint4*>(sWq)[idx] = src[idx];
    const int per_row = DH / 8;
    for (int idx = threadIdx.x; idx < d * per_row; idx += blockDim.x) {
      const int o = idx / per_row, c8 = (idx % per_row) * 8;
      const uint4 v = *reinterpret_cast<const uint4*>(w.Wo2 + (size_t)o * d + h * DH + c8);
      const __nv_bfloat16* e = reinterpret_cast<const __nv_bfloat16*>(&v);
#pragma unroll
      for (int j = 0; j < 8; ++j) sWo[(size_t)(c8 + j) * d + o] = e[j];
    }
  }
  __syncthreads();
  for (int c = warp; c < DH; c += (blockDim.x >> 5)) {
    float a = 0.f;
    for (int i = lane; i < d; i += 32) a += w.ln_b[i] * __bfloat162float(sWq[(size_t)c * d + i]);
    a = warp_sum(a);
    if (lane == 0) swb[c] = a + w.bq2[h * DH + c];
  }
  const float scale = rsqrtf((float)DH);
  // four memory tokens at a time: a weight pair read from shared memory serves 8 outputs
  for (int row0 = blockIdx.y * XF_RB; row0 < rows; row0 += gridDim.y * XF_RB) {
    __syncthreads();
    for (int idx = threadIdx.x; idx < 2 * DH * XF_RB; idx += blockDim.x) {
      const int rr = idx % XF_RB, c = (idx / XF_RB) % DH, which = idx / (XF_RB * DH);
      const int row = row0 + rr;
      sk[idx] = row < rows ? kv[(size_t)row * ldkv + (size_t)layer * 2 * d + (size_t)which * d + h * DH + c] : 0.f;
    }
    __syncthreads();
    const float4* sk4 = reinterpret_cast<const float4*>(sk);       // [k | v][c] -> the 4 rows' values
    for (int i2 = threadIdx.x; i2 < d / 2; i2 += blockDim.x) {
      float aq[XF_RB][2], au[XF_RB][2];
#pragma unroll
      for (int rr = 0; rr < XF_RB; ++rr) { aq[rr][0] = aq[rr][1] = au[rr][0] = au[rr][1] = 0.f; }
      for (int c = 0; c < DH; ++c) {
        const float2 wq = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(sWq + (size_t)c * d + 2 * i2));
        const float2 wo = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(sWo + (size_t)c * d + 2 * i2));
        const float4 k4 = sk4[c], v4 = sk4[DH + c];
        const float kk[4] = {k4.x, k4.y, k4.z, k4.w}, vv[4] = {v4.x, v4.y, v4.z, v4.w};
#pragma unroll
        for (int rr = 0; rr < XF_RB; ++rr) {
          aq[rr][0] += wq.x * kk[rr]; aq[rr][1] += wq.y * kk[rr];
          au[rr][0] += wo.x * vv[rr]; au[rr][1] += wo.y * vv[rr];
        }
      }
      const int i = 2 * i2;
      const float g0 = scale * w.ln_g[i], g1 = scale * w.ln_g[i + 1];
#pragma unroll
      for (int rr = 0; rr < XF_RB; ++rr) {
        const int row = row0 + rr;
        if (row < rows) {
          const size_t base = ((size_t)row * L + layer) * heads * d;
          *reinterpret_cast<uint32_t*>(kq + base + (size_t)h * d + i) = pack_bf16(aq[rr][0] * g0, aq[rr][1] * g1);
          ut[base + ((size_t)(h >> 1) * d + i) * 2 + (h & 1)] = __float2bfloat16_rn(au[rr][0]);
          ut[base + ((size_t)(h >> 1) * d + i + 1) * 2 + (h & 1)] = __float2bfloat16_rn(au[rr][1]);
        }
      }
    }
    if (warp < XF_RB && row0 + warp < rows) {
      float a = 0.f;
      for (int c = lane; c < DH; c += 32) a += sk[c * XF_RB + warp] * swb[c];
      a = warp_sum(a);
      if (lane == 0) cc[((size_t)(row0 + warp) * L + layer) * heads + h] = a * scale;
    }
  }
}

__device__ __forceinline__ uint32_t xf_ldg32(const __nv_bfloat16* p) { return __ldg(reinterpret_cast<const unsigned int*>(p)); }

// One block per candidate (H <= 16 token rows of width D), 4 warps.
//   1  xhat = LayerNorm without affine of the candidate's rows, bf16, into shared memory (warp w: rows 4w..4w+3)
//   2  partial scores of warp w over its quarter of the D input columns, summed through shared memory
//   3  softmax over the memory tokens per (row, head) -> P [16 x 32] bf16
//   4  warp w: output columns [w D/4, (w+1) D/4) = P . U, + bo2, added to the residual stream in place
// Every phase issues all of its global loads before it uses the first of them: a block is a chain of a
// few memory round trips, and with four warps nothing else would hide them.
template <int D>
__global__ void __launch_bounds__(XF_THREADS)
xattn_fold_kernel(float* __restrict__ x, XfoldTables tb, const float* __restrict__ bo2, CandMap cm, int H, int heads,
                  int To, int layer, int L, int Tsteps) {
  pdl_trigger();
  pdl_wait();
  constexpr int LDA = D + 8;
  constexpr int LDP = XF_MAXN + 8;
  constexpr int V = D / 128;
  __shared__ __align__(16) __nv_bfloat16 sA[16 * LDA];
  __shared__ float sS[4][16][XF_MAXN];
  __shared__ __align__(16) __nv_bfloat16 sP[16 * LDP];
  const int n = blockIdx.x;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, tg = lane & 3;
  const int b = n / cm.C, cnd = n % cm.C;
  int tau = cm.t[b] - cm.koff - cnd;
  tau = max(0, min(Tsteps - 1, tau));
  const int item = item_of(cm.item, b);
  const int NK = 1 + To, NKH = NK * heads;
  const size_t tok_stride = (size_t)L * heads * D;      // kq / ut elements per memory token
  const size_t lay_off = (size_t)layer * heads * D;
  float* xc = x + (size_t)n * H * D;

  // ---- 1: LayerNorm statistics, normalised rows to shared memory
  for (int i = threadIdx.x; i < 16 * LDP / 2; i += XF_THREADS) reinterpret_cast<uint32_t*>(sP)[i] = 0u;
#pragma unroll 1
  for (int rb = 0; rb < 4; rb += 2) {          // two rows per pass: all of their loads are in flight together
    float4 v[2][V];
#pragma unroll
    for (int rr = 0; rr < 2; ++rr) {
      const int r = min(4 * warp + rb + rr, H - 1);
#pragma unroll
      for (int j = 0; j < V; ++j) v[rr][j] = reinterpret_cast<const float4*>(xc + (size_t)r * D)[j * 32 + lane];
    }
#pragma unroll
    for (int rr = 0; rr < 2; ++rr) {
      const int r = 4 * warp + rb + rr;
      float s = 0.f;
#pragma unroll
      for (int j = 0; j < V; ++j) s += v[rr][j].x + v[rr][j].y + v[rr][j].z + v[rr][j].w;
      const float mean = warp_sum(s) / D;
      float q = 0.f;
#pragma unroll
      for (int j = 0; j < V; ++j) {
        float4& e = v[rr][j];
        e.x -= mean; e.y -= mean; e.z -= mean; e.w -= mean;
        q += e.x * e.x + e.y * e.y + e.z * e.z + e.w * e.w;
      }
      const float rstd = r < H ? rsqrtf(warp_sum(q) / D + 1e-5f) : 0.f;      // rows past H enter the products as zeros
#pragma unroll
      for (int j = 0; j < V; ++j) {
        uint2 pk2;
        pk2.x = pack_bf16(v[rr][j].x * rstd, v[rr][j].y * rstd);
        pk2.y = pack_bf16(v[rr][j].z * rstd, v[rr][j].w * rstd);
        *reinterpret_cast<uint2*>(sA + r * LDA + (j * 32 + lane) * 4) = pk2;
      }
    }
  }
  __syncthreads();

  // ---- 2: scores, k steps [warp * D/64, (warp + 1) * D/64)
  {
    const __nv_bfloat16* pk[4];
    uint32_t live[4];
#pragma unroll
    for (int nt = 0; nt < 4; ++nt) {
      const int nn = min(8 * nt + g, NKH - 1);            // lanes past the last (token, head) read a valid row, masked below
      live[nt] = 8 * nt + g < NKH ? 0xffffffffu : 0u;
      const int j = nn / heads, h = nn % heads;
      pk[nt] = (j == 0 ? tb.kq_time + (size_t)tau * tok_stride : tb.kq_obs + ((size_t)item * To + (j - 1)) * tok_stride) + lay_off +
               (size_t)h * D + (size_t)warp * (D / 4) + 2 * tg;
    }
    float sc[4][4];
#pragma unroll
    for (int nt = 0; nt < 4; ++nt) { sc[nt][0] = sc[nt][1] = sc[nt][2] = sc[nt][3] = 0.f; }
    constexpr int KSW = D / 64;
    constexpr int KB = KSW < 4 ? KSW : 4;
#pragma unroll
    for (int kb = 0; kb < KSW; kb += KB) {
      uint32_t bq[KB][4][2];
#pragma unroll
      for (int kk = 0; kk < KB; ++kk)
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) {
          if (8 * nt < NKH) {
            const __nv_bfloat16* p = pk[nt] + (kb + kk) * 16;
            bq[kk][nt][0] = xf_ldg32(p);
            bq[kk][nt][1] = xf_ldg32(p + 8);
          }
        }
#pragma unroll
      for (int kk = 0; kk < KB; ++kk) {
        const int ks = warp * KSW + kb + kk;
        uint32_t a[4];
        const __nv_bfloat16* ar = sA + g * LDA + ks * 16 + 2 * tg;
        a[0] = *reinterpret_cast<const uint32_t*>(ar);
        a[1] = *reinterpret_cast<const uint32_t*>(ar + 8 * LDA);
        a[2] = *reinterpret_cast<const uint32_t*>(ar + 8);
        a[3] = *reinterpret_cast<const uint32_t*>(ar + 8 * LDA + 8);
#pragma unroll
        for (int nt = 0; nt < 4; ++nt)
          if (8 * nt < NKH) mma_bf16_16816(sc[nt], a, bq[kk][nt][0] & live[nt], bq[kk][nt][1] & live[nt]);
      }
    }
#pragma unroll
    for (int nt = 0; nt < 4; ++nt) {
      sS[warp][g][8 * nt + 2 * tg] = sc[nt][0]; sS[warp][g][8 * nt + 2 * tg + 1] = sc[nt][1];
      sS[warp][g + 8][8 * nt + 2 * tg] = sc[nt][2]; sS[warp][g + 8][8 * nt + 2 * tg + 1] = sc[nt][3];
    }
  }
  __syncthreads();

  // ---- 3: softmax over the NK memory tokens for every (row, head)
  for (int idx = threadIdx.x; idx < 16 * heads; idx += XF_THREADS) {
    const int r = idx / heads, h = idx % heads;
    float s[XF_MAXNK];
#pragma unroll
    for (int j = 0; j < XF_MAXNK; ++j) {
      if (j < NK) {
        const float* cp = (j == 0 ? tb.c_time + (size_t)tau * L * heads : tb.c_obs + ((size_t)item * To + (j - 1)) * L * heads) +
                          (size_t)layer * heads;
        s[j] = __ldg(cp + h);
      }
    }
    float m = -INFINITY;
#pragma unroll
    for (int j = 0; j < XF_MAXNK; ++j) {
      if (j < NK) {
        const int nn = j * heads + h;
        s[j] += sS[0][r][nn] + sS[1][r][nn] + sS[2][r][nn] + sS[3][r][nn];
        m = fmaxf(m, s[j]);
      }
    }
    float l = 0.f;
#pragma unroll
    for (int j = 0; j < XF_MAXNK; ++j)
      if (j < NK) { s[j] = __expf(s[j] - m); l += s[j]; }
    const float inv = 1.0f / l;
#pragma unroll
    for (int j = 0; j < XF_MAXNK; ++j)
      if (j < NK) sP[r * LDP + j * heads + h] = __float2bfloat16_rn(s[j] * inv);
  }
  __syncthreads();

  // ---- 4: P . U + bo2 into the residual stream, four 8-column tiles at a time
  {
    uint32_t pa[2][4];
#pragma unroll
    for (int k2 = 0; k2 < 2; ++k2) {
      const __nv_bfloat16* ar = sP + g * LDP + k2 * 16 + 2 * tg;
      pa[k2][0] = *reinterpret_cast<const uint32_t*>(ar);
      pa[k2][1] = *reinterpret_cast<const uint32_t*>(ar + 8 * LDP);
      pa[k2][2] = *reinterpret_cast<const uint32_t*>(ar + 8);
      pa[k2][3] = *reinterpret_cast<const uint32_t*>(ar + 8 * LDP + 8);
    }
    const __nv_bfloat16* pu[2][2];
    uint32_t ulive[2][2];
#pragma unroll
    for (int k2 = 0; k2 < 2; ++k2)
#pragma unroll
      for (int rg = 0; rg < 2; ++rg) {
        const int n0 = 16 * k2 + 8 * rg + 2 * tg;
        ulive[k2][rg] = n0 < NKH ? 0xffffffffu : 0u;
        const int nn = min(n0, NKH - 2);
        const int j = nn / heads, h = nn % heads;
        pu[k2][rg] = (j == 0 ? tb.ut_time + (size_t)tau * tok_stride : tb.ut_obs + ((size_t)item * To + (j - 1)) * tok_stride) + lay_off +
                     ((size_t)(h >> 1) * D + g) * 2;
      }
    const bool row0 = g < H, row1 = g + 8 < H;
    float* x0 = xc + (size_t)(row0 ? g : 0) * D;
    float* x1 = xc + (size_t)(row1 ? g + 8 : 0) * D;
    constexpr int NTB = 4;
#pragma unroll 1
    for (int o_base = warp * (D / 4); o_base < (warp + 1) * (D / 4); o_base += 8 * NTB) {
      uint32_t bu[NTB][2][2];
      float2 xv[NTB][2], bb[NTB];
#pragma unroll
      for (int nt = 0; nt < NTB; ++nt) {
        const int o = (o_base + 8 * nt) * 2;
#pragma unroll
        for (int k2 = 0; k2 < 2; ++k2) {
          if (16 * k2 < NKH) {
            bu[nt][k2][0] = xf_ldg32(pu[k2][0] + o);
            bu[nt][k2][1] = xf_ldg32(pu[k2][1] + o);
          }
        }
        const int col = o_base + 8 * nt + 2 * tg;
        xv[nt][0] = *reinterpret_cast<const float2*>(x0 + col);
        xv[nt][1] = *reinterpret_cast<const float2*>(x1 + col);
        bb[nt] = __ldg(reinterpret_cast<const float2*>(bo2 + col));
      }
#pragma unroll
      for (int nt = 0; nt < NTB; ++nt) {
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int k2 = 0; k2 < 2; ++k2)
          if (16 * k2 < NKH) mma_bf16_16816(acc, pa[k2], bu[nt][k2][0] & ulive[k2][0], bu[nt][k2][1] & ulive[k2][1]);
        const int col = o_base + 8 * nt + 2 * tg;
        if (row0) *reinterpret_cast<float2*>(x0 + col) = make_float2(xv[nt][0].x + acc[0] + bb[nt].x, xv[nt][0].y + acc[1] + bb[nt].y);
        if (row1) *reinterpret_cast<float2*>(x1 + col) = make_float2(xv[nt][1].x + acc[2] + bb[nt].x, xv[nt][1].y + acc[3] + bb[nt].y);
      }
    }
  }
}

}  // namespace tsdp
