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
//   kq [row][layer][heads][d]           one contiguous row of d values per (memory token, head)
//   ut [row][layer][heads/2][d][2]      heads in pairs: word (q, o) holds u of heads 2q and 2q+1 at output column o,
//                                       which is one B-fragment register of the second product
//   cc [row][layer][heads]  fp32
#pragma once
#include "common.cuh"
#include "net_kernels.cuh"

namespace tsdp {

constexpr int XF_THREADS = 256;
constexpr int XF_WARPS = XF_THREADS / 32;
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

__device__ __forceinline__ void xf_cp16(void* smem_dst, const void* gsrc) {
  const uint32_t d = (uint32_t)__cvta_generic_to_shared(smem_dst);
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void xf_add_bf16x4(float4& a, const uint2 d) {
  const float2 lo = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&d.x));
  const float2 hi = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&d.y));
  a.x += lo.x; a.y += lo.y; a.z += hi.x; a.w += hi.y;
}
// fp32 arithmetic two values at a time (packed fp32 pipe; each component rounded as the scalar operation would be)
__device__ __forceinline__ float2 xf_lo(const float4& a) { return make_float2(a.x, a.y); }
__device__ __forceinline__ float2 xf_hi(const float4& a) { return make_float2(a.z, a.w); }
__device__ __forceinline__ float4 xf_join(float2 lo, float2 hi) { return make_float4(lo.x, lo.y, hi.x, hi.y); }
__device__ __forceinline__ float2 xf_dup(float v) { return make_float2(v, v); }
__device__ __forceinline__ void xf_cp_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void xf_cp_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// Shared memory of one block: xhat [16][D+8] bf16 | kq rows [NKH][D+8] bf16 (both dead after the scores: the product
// P . U [16][D+8] fp32 is then laid over the two) | u rows [NKH/2][D+8] words | partial scores [4][16][32] fp32 |
// P [16][40] bf16.
__host__ __device__ constexpr size_t xf_region_bytes(int D, int nkh) {
  const size_t k = (size_t)nkh * (D + 8) * 2, t = (size_t)16 * (D + 8) * 2;     // xhat + region >= [16][D+8] fp32
  return k > t ? k : t;
}
__host__ __device__ constexpr size_t xf_smem_bytes(int D, int nkh) {
  return (size_t)16 * (D + 8) * 2 + xf_region_bytes(D, nkh) + (size_t)(nkh / 2) * (D + 8) * 4 + (size_t)4 * 16 * XF_MAXN * 4 +
         (size_t)16 * (XF_MAXN + 8) * 2;
}

// One block per candidate (H <= 16 token rows of width D), 8 warps.
//   0  the candidate's kq and u rows start their way into shared memory (cp.async, 16 bytes per lane: a
//      lane-by-lane gather of tensor-core fragments from global memory is bound by the L1 tag rate)
//   1  xhat = LayerNorm without affine of the candidate's rows, bf16, into shared memory (warp w: rows 2w, 2w+1)
//   2  partial scores: warp w covers a quarter of the D input columns for two of the 8-wide score tiles
//   3  softmax over the memory tokens per (row, head) -> P [16 x 32] bf16
//   4  warp w: output columns [w D/8, (w+1) D/8) of P . U for all 16 rows -> shared memory (fp32)
//   5  warp w again owns rows 2w, 2w+1, whose residual values (stream + delta) are still in its registers from
//      phase 1: adds the product and bo2, writes the stream back in full 16-byte lanes, and applies the LayerNorm in
//      front of the MLP with warp-level statistics -> ln3_out (bf16)
// `delta` is the output of the self-attention projection (bf16, bias included), which this kernel adds to the
// residual stream before anything else: that GEMM then writes 2 bytes per element instead of doing an fp32
// read-modify-write of the stream.
template <int D>
__global__ void __launch_bounds__(XF_THREADS, 3)
xattn_fold_kernel(float* __restrict__ x, const __nv_bfloat16* __restrict__ delta, XfoldTables tb, const float* __restrict__ bo2,
                  const float* __restrict__ ln3_g, const float* __restrict__ ln3_b, __nv_bfloat16* __restrict__ ln3_out, CandMap cm,
                  int H, int heads, int To, int layer, int L, int Tsteps) {
  pdl_trigger();
  pdl_wait();
  constexpr int LDA = D + 8;               // bf16 elements per row of xhat and of the kq rows
  constexpr int LDU = D + 8;               // words per row of the u rows
  constexpr int LDP = XF_MAXN + 8;
  constexpr int V = D / 128;
  extern __shared__ __align__(16) unsigned char xf_smem[];
  const int NK = 1 + To, NKH = NK * heads;
  __nv_bfloat16* sA = reinterpret_cast<__nv_bfloat16*>(xf_smem);
  unsigned char* region = xf_smem + (size_t)16 * LDA * 2;
  __nv_bfloat16* sK = reinterpret_cast<__nv_bfloat16*>(region);
  uint32_t* sU = reinterpret_cast<uint32_t*>(region + xf_region_bytes(D, NKH));
  float* sS = reinterpret_cast<float*>(sU + (size_t)(NKH / 2) * LDU);      // [4][16][XF_MAXN]
  __nv_bfloat16* sP = reinterpret_cast<__nv_bfloat16*>(sS + 4 * 16 * XF_MAXN);
  const int n = blockIdx.x;
  if (n >= cand_count(cm, gridDim.x)) return;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, tg = lane & 3;
  int b, cnd;
  cand_decode(cm, n, b, cnd);
  int tau = cm.t[b] - cm.koff - cnd;
  tau = max(0, min(Tsteps - 1, tau));
  const int item = item_of(cm.item, b);
  const size_t tok_stride = (size_t)L * heads * D;      // kq / ut elements per memory token
  const size_t lay_off = (size_t)layer * heads * D;
  float* xc = x + (size_t)n * H * D;
  const __nv_bfloat16* dc = delta + (size_t)n * H * D;

  // ---- 0: tables of this candidate's memory tokens, one row per warp at a time
  {
    const int hp = heads >> 1;
    for (int row = warp; row < NKH; row += XF_WARPS) {
      const int jt = row / heads, h = row - jt * heads;
      const __nv_bfloat16* sr = (jt == 0 ? tb.kq_time + (size_t)tau * tok_stride : tb.kq_obs + ((size_t)item * To + (jt - 1)) * tok_stride) +
                                lay_off + (size_t)h * D;
      __nv_bfloat16* dr = sK + (size_t)row * LDA;
#pragma unroll
      for (int ch = 0; ch < D / 256; ++ch) xf_cp16(dr + (ch * 32 + lane) * 8, sr + (ch * 32 + lane) * 8);
      if (D % 256 && lane < (D % 256) / 8) xf_cp16(dr + (D / 256 * 32 + lane) * 8, sr + (D / 256 * 32 + lane) * 8);
    }
    xf_cp_commit();
    for (int row = warp; row < NKH / 2; row += XF_WARPS) {
      const int jt = row / hp, q = row - jt * hp;
      const __nv_bfloat16* sr = (jt == 0 ? tb.ut_time + (size_t)tau * tok_stride : tb.ut_obs + ((size_t)item * To + (jt - 1)) * tok_stride) +
                                lay_off + (size_t)q * D * 2;
      uint32_t* dr = sU + (size_t)row * LDU;
#pragma unroll
      for (int ch = 0; ch < D / 128; ++ch) xf_cp16(dr + (ch * 32 + lane) * 4, sr + (ch * 32 + lane) * 8);
    }
    xf_cp_commit();
  }

  // ---- 1: LayerNorm statistics, normalised rows to shared memory
  for (int i = threadIdx.x; i < 16 * LDP / 2; i += XF_THREADS) reinterpret_cast<uint32_t*>(sP)[i] = 0u;
  float4 xr[2][V];                             // rows 2 warp, 2 warp + 1 of the stream with delta added: kept until phase 5
  // the score constants this thread needs in phase 3: in flight from here on
  float cst[XF_MAXNK];
  {
    const int h = threadIdx.x % heads;
#pragma unroll
    for (int j = 0; j < XF_MAXNK; ++j) {
      cst[j] = 0.f;
      if (j < NK && threadIdx.x < 16 * heads) {
        const float* cp = (j == 0 ? tb.c_time + (size_t)tau * L * heads : tb.c_obs + ((size_t)item * To + (j - 1)) * L * heads) +
                          (size_t)layer * heads;
        cst[j] = __ldg(cp + h);
      }
    }
  }
  {                                            // two rows per warp: all of their loads are in flight together
    float4 v[2][V];
#pragma unroll
    for (int rr = 0; rr < 2; ++rr) {
      const int r = min(2 * warp + rr, H - 1);
#pragma unroll
      for (int j = 0; j < V; ++j) v[rr][j] = reinterpret_cast<const float4*>(xc + (size_t)r * D)[j * 32 + lane];
    }
    uint2 dv[2][V];
#pragma unroll
    for (int rr = 0; rr < 2; ++rr) {
      const int r = min(2 * warp + rr, H - 1);
#pragma unroll
      for (int j = 0; j < V; ++j) dv[rr][j] = reinterpret_cast<const uint2*>(dc + (size_t)r * D)[j * 32 + lane];
    }
#pragma unroll
    for (int rr = 0; rr < 2; ++rr)
#pragma unroll
      for (int j = 0; j < V; ++j) { xf_add_bf16x4(v[rr][j], dv[rr][j]); xr[rr][j] = v[rr][j]; }
#pragma unroll
    for (int rr = 0; rr < 2; ++rr) {
      const int r = 2 * warp + rr;
      float2 s2 = make_float2(0.f, 0.f);
#pragma unroll
      for (int j = 0; j < V; ++j) s2 = __fadd2_rn(s2, __fadd2_rn(xf_lo(v[rr][j]), xf_hi(v[rr][j])));
      const float mean = warp_sum(s2.x + s2.y) / D;
      const float2 nm = xf_dup(-mean);
      float2 q2 = make_float2(0.f, 0.f);
      float2 lo[V], hi[V];
#pragma unroll
      for (int j = 0; j < V; ++j) {
        lo[j] = __fadd2_rn(xf_lo(v[rr][j]), nm); hi[j] = __fadd2_rn(xf_hi(v[rr][j]), nm);
        q2 = __ffma2_rn(lo[j], lo[j], q2); q2 = __ffma2_rn(hi[j], hi[j], q2);
      }
      const float rstd = r < H ? rsqrtf(warp_sum(q2.x + q2.y) / D + 1e-5f) : 0.f;      // rows past H enter the products as zeros
      const float2 rs2 = xf_dup(rstd);
#pragma unroll
      for (int j = 0; j < V; ++j) {
        const float2 a = __fmul2_rn(lo[j], rs2), b = __fmul2_rn(hi[j], rs2);
        uint2 pk2;
        pk2.x = pack_bf16(a.x, a.y);
        pk2.y = pack_bf16(b.x, b.y);
        *reinterpret_cast<uint2*>(sA + r * LDA + (j * 32 + lane) * 4) = pk2;
      }
    }
  }
  xf_cp_wait<1>();                             // this thread's kq chunks have landed
  __syncthreads();

  // ---- 2: scores.  Warp w takes quarter (w & 3) of the D input columns and the score tiles 2 (w >> 2), 2 (w >> 2) + 1;
  //         the four partial sums of a score are added in a fixed order in phase 3 (no atomics: same bits every run).
  //         Score columns past the last (token, head) are computed on a repeated row and never read.
  {
    constexpr int KSW = D / 64;
    const int kq4 = warp & 3, nh = warp >> 2;
    float sc[2][4];
#pragma unroll
    for (int u = 0; u < 2; ++u) { sc[u][0] = sc[u][1] = sc[u][2] = sc[u][3] = 0.f; }
    if (16 * nh < NKH) {
      // ldmatrix addresses: A rows l & 15 at column 8 (l >> 4); B rows 16 nh + (l & 7) + 8 (l >> 4) at column 8 ((l >> 3) & 1)
      const __nv_bfloat16* pa_l = sA + (lane & 15) * LDA + kq4 * (D / 4) + 8 * (lane >> 4);
      const __nv_bfloat16* pb_l = sK + (size_t)min(16 * nh + (lane & 7) + 8 * (lane >> 4), NKH - 1) * LDA + kq4 * (D / 4) +
                                  8 * ((lane >> 3) & 1);
#pragma unroll
      for (int kk = 0; kk < KSW; ++kk) {
        uint32_t a[4], b[4];
        ldmatrix_x4(a, pa_l + kk * 16);
        ldmatrix_x4(b, pb_l + kk * 16);
        mma_bf16_16816(sc[0], a, b[0], b[1]);
        mma_bf16_16816(sc[1], a, b[2], b[3]);
      }
    }
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      float* s0 = sS + ((size_t)kq4 * 16 + g) * XF_MAXN + 8 * (2 * nh + u) + 2 * tg;
      s0[0] = sc[u][0]; s0[1] = sc[u][1];
      s0[8 * XF_MAXN] = sc[u][2]; s0[8 * XF_MAXN + 1] = sc[u][3];
    }
  }
  __syncthreads();

  // ---- 3: softmax over the NK memory tokens for every (row, head)
  if (threadIdx.x < 16 * heads) {              // heads <= 16: one (row, head) per thread
    const int idx = threadIdx.x;
    const int r = idx / heads, h = idx % heads;
    float s[XF_MAXNK];
#pragma unroll
    for (int j = 0; j < XF_MAXNK; ++j) s[j] = cst[j];
    float m = -INFINITY;
#pragma unroll
    for (int j = 0; j < XF_MAXNK; ++j) {
      if (j < NK) {
        const int nn = j * heads + h;
        s[j] += ((sS[(0 * 16 + r) * XF_MAXN + nn] + sS[(1 * 16 + r) * XF_MAXN + nn]) + sS[(2 * 16 + r) * XF_MAXN + nn]) +
                sS[(3 * 16 + r) * XF_MAXN + nn];
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
  xf_cp_wait<0>();                             // this thread's u chunks have landed
  __syncthreads();                             // also: every warp is done with the normalised rows and the kq rows, whose memory the product reuses

  // ---- 4: P . U for all 16 rows, warp w the output columns [w D/8, (w+1) D/8), into shared memory over the
  //         (now dead) normalised rows and kq rows
  constexpr int LDO = D + 8;                   // fp32 words per row of the product
  float* sO = reinterpret_cast<float*>(xf_smem);
  {
    uint32_t pa[2][4];
#pragma unroll
    for (int k2 = 0; k2 < 2; ++k2) ldmatrix_x4(pa[k2], sP + (lane & 15) * LDP + k2 * 16 + 8 * (lane >> 4));
    // B fragment (k2, rg) of a lane: memory-token/head pair row 8 k2 + 4 rg + tg of the u rows
    const uint32_t* pu[2][2];
    uint32_t ulive[2][2];
#pragma unroll
    for (int k2 = 0; k2 < 2; ++k2)
#pragma unroll
      for (int rg = 0; rg < 2; ++rg) {
        const int pr = 8 * k2 + 4 * rg + tg;
        ulive[k2][rg] = 2 * pr < NKH ? 0xffffffffu : 0u;
        pu[k2][rg] = sU + (size_t)min(pr, NKH / 2 - 1) * LDU + g;
      }
    const int o_base = warp * (D / XF_WARPS);
#pragma unroll
    for (int nt = 0; nt < D / (8 * XF_WARPS); ++nt) {
      float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int k2 = 0; k2 < 2; ++k2)
        if (16 * k2 < NKH)
          mma_bf16_16816(acc, pa[k2], pu[k2][0][o_base + 8 * nt] & ulive[k2][0], pu[k2][1][o_base + 8 * nt] & ulive[k2][1]);
      *reinterpret_cast<float2*>(sO + g * LDO + o_base + 8 * nt + 2 * tg) = make_float2(acc[0], acc[1]);
      *reinterpret_cast<float2*>(sO + (g + 8) * LDO + o_base + 8 * nt + 2 * tg) = make_float2(acc[2], acc[3]);
    }
  }
  // bo2 of this lane's columns: in flight across the barrier
  float4 bb[V];
#pragma unroll
  for (int j = 0; j < V; ++j) bb[j] = __ldg(reinterpret_cast<const float4*>(bo2) + j * 32 + lane);
  __syncthreads();

  // ---- 5: rows 2 warp, 2 warp + 1: stream + delta (registers) + product + bo2 -> the stream; LayerNorm -> ln3_out
  {
#pragma unroll
    for (int rr = 0; rr < 2; ++rr) {
      const int r = 2 * warp + rr;
#pragma unroll
      for (int j = 0; j < V; ++j) {
        const float4 t = *reinterpret_cast<const float4*>(sO + r * LDO + (j * 32 + lane) * 4);
        float4& e = xr[rr][j];
        e = xf_join(__fadd2_rn(xf_lo(e), __fadd2_rn(xf_lo(t), xf_lo(bb[j]))), __fadd2_rn(xf_hi(e), __fadd2_rn(xf_hi(t), xf_hi(bb[j]))));
        if (r < H) reinterpret_cast<float4*>(xc + (size_t)r * D)[j * 32 + lane] = e;
      }
    }
    float4 gg[V], be[V];
#pragma unroll
    for (int j = 0; j < V; ++j) {
      gg[j] = __ldg(reinterpret_cast<const float4*>(ln3_g) + j * 32 + lane);
      be[j] = __ldg(reinterpret_cast<const float4*>(ln3_b) + j * 32 + lane);
    }
    __nv_bfloat16* oc = ln3_out + (size_t)n * H * D;
#pragma unroll
    for (int rr = 0; rr < 2; ++rr) {
      const int r = 2 * warp + rr;
      float2 s2 = make_float2(0.f, 0.f);
#pragma unroll
      for (int j = 0; j < V; ++j) s2 = __fadd2_rn(s2, __fadd2_rn(xf_lo(xr[rr][j]), xf_hi(xr[rr][j])));
      const float mean = warp_sum(s2.x + s2.y) / D;
      const float2 nm = xf_dup(-mean);
      float2 q2 = make_float2(0.f, 0.f);
      float2 lo[V], hi[V];
#pragma unroll
      for (int j = 0; j < V; ++j) {
        lo[j] = __fadd2_rn(xf_lo(xr[rr][j]), nm); hi[j] = __fadd2_rn(xf_hi(xr[rr][j]), nm);
        q2 = __ffma2_rn(lo[j], lo[j], q2); q2 = __ffma2_rn(hi[j], hi[j], q2);
      }
      const float2 rs2 = xf_dup(rsqrtf(warp_sum(q2.x + q2.y) / D + 1e-5f));
      if (r < H) {
#pragma unroll
        for (int j = 0; j < V; ++j) {
          const float2 a = __ffma2_rn(__fmul2_rn(lo[j], rs2), xf_lo(gg[j]), xf_lo(be[j]));
          const float2 b = __ffma2_rn(__fmul2_rn(hi[j], rs2), xf_hi(gg[j]), xf_hi(be[j]));
          uint2 o2;
          o2.x = pack_bf16(a.x, a.y);
          o2.y = pack_bf16(b.x, b.y);
          reinterpret_cast<uint2*>(oc + (size_t)r * D)[j * 32 + lane] = o2;
        }
      }
    }
  }
}

}  // namespace tsdp
