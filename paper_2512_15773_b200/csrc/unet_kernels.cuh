// Kernels of the 1-D temporal conv UNet around its convolutions.  Activations are channels-last and
// zero-padded along the sequence: a tensor of L positions and C channels of n candidates is stored as
// [n, L + 4, C] with two zero rows before and after the L valid ones.  In that layout the im2col
// matrix of a kernel-5 "same" convolution is a VIEW: row (n, l) starts at element ((n (L+4) + l) C)
// and is 5 C elements long (rows overlap), so every convolution runs on the tensor-core GEMM through a
// tensor map whose row pitch is C instead of 5 C.  Its output row r = n (L+4) + l is valid for l < L.
// The kernels here write only valid rows, so the padding rows stay zero for the lifetime of a buffer.
#pragma once
#include "common.cuh"
#include "net_kernels.cuh"
#include "dit_kernels.cuh"

namespace tsdp {

__device__ __forceinline__ float mish_f(float v) {
  const float sp = v > 20.f ? v : log1pf(expf(v));       // softplus
  return v * tanhf(sp);
}

__global__ void mish_kernel(const float* in, float* out, long long n) {
  pdl_trigger();
  pdl_wait();
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) out[i] = mish_f(in[i]);
}

// Input projection: X[n, l + 2, :] = x[n, l, :] W_in + b_in   (pointwise, A -> C channels).
template <typename T>
__global__ void unet_embed_kernel(CandMap cm, const float* __restrict__ W_in, const float* __restrict__ b_in,
                                  T* __restrict__ X, int H, int A, int C) {
  pdl_trigger();
  pdl_wait();
  const int row = blockIdx.x;                      // n * H + l
  const int n = row / H, l = row % H;
  if (n >= cand_count(cm, gridDim.x / H)) return;
  int b, c;
  cand_decode(cm, n, b, c);
  const float* x = cm.xin + b * cm.x_stride_b + (long long)c * H * A + (long long)l * A;
  T* o = X + ((size_t)n * (H + 4) + l + 2) * C;
  for (int col = threadIdx.x; col < C; col += blockDim.x) {
    float v = b_in[col];
    for (int a = 0; a < A; ++a) v += x[a] * W_in[a * C + col];
    o[col] = from_f<T>(v);
  }
}

// GroupNorm + Mish (+ FiLM) (+ residual) over one (candidate, group); Y is the fp32 convolution output
// [n (L+4) rows, C], valid rows l < L.
//   v = Mish(GN(Y)) ; v = scale v + bias (film != null) ; v += residual ; dst[n, l+2, coff + c] = v
// FiLM vectors of candidate n: film_time[tau(n)] + film_obs[item(n)], this block's scale at column foff,
// its bias at foff + C.  Residual: res_t (same type as dst, padded [n, L+4, res_pitch], channels 0..C-1) or
// res_f (fp32 rows in the padded indexing n (L+4) + l + 2, pitch C); at most one of them.
template <typename T>
__global__ void __launch_bounds__(256)
gn_mish_kernel(const float* __restrict__ Y, const float* __restrict__ gam, const float* __restrict__ bet, int groups,
               const float* __restrict__ film_time, const float* __restrict__ film_obs, int F, int foff, CandMap cm,
               int Tsteps, const T* __restrict__ res_t, int res_pitch, const float* __restrict__ res_f,
               T* __restrict__ dst, int dst_pitch, int coff, int L, int C, int n_split, long long split_stride) {
  pdl_trigger();
  pdl_wait();
  __shared__ float red[2][8];
  // Y may arrive as n_split partial sums of the convolution's reduction, split_stride elements apart: added here in
  // the order of the parts, whichever CTA produced which
  auto y_at = [&](size_t idx) {
    if (n_split <= 1) return Y[idx];
    float part[8];                               // at most 8 parts: all loads in flight together, added in order
#pragma unroll
    for (int sp = 0; sp < 8; ++sp) part[sp] = sp < n_split ? Y[idx + (size_t)sp * (size_t)split_stride] : 0.f;
    float v = part[0];
#pragma unroll
    for (int sp = 1; sp < 8; ++sp) if (sp < n_split) v += part[sp];
    return v;
  };
  const int n = blockIdx.x / groups, grp = blockIdx.x % groups;
  if (n >= cand_count(cm, gridDim.x / groups)) return;
  const int Cg = C / groups, Lp = L + 4;
  const int cnt = L * Cg;
  const size_t y0 = (size_t)n * Lp * C + (size_t)grp * Cg;
  float s = 0.f, q = 0.f;
  for (int i = threadIdx.x; i < cnt; i += blockDim.x) {
    const float v = y_at(y0 + (size_t)(i / Cg) * C + (i % Cg));
    s += v; q += v * v;
  }
  s = warp_sum(s); q = warp_sum(q);
  if ((threadIdx.x & 31) == 0) { red[0][threadIdx.x >> 5] = s; red[1][threadIdx.x >> 5] = q; }
  __syncthreads();
  float ts = 0.f, tq = 0.f;
  for (int w = 0; w < (int)(blockDim.x >> 5); ++w) { ts += red[0][w]; tq += red[1][w]; }
  const float mean = ts / cnt;
  const float rstd = rsqrtf(fmaxf(tq / cnt - mean * mean, 0.f) + 1e-5f);
  const float *ft = nullptr, *fo = nullptr;
  if (film_time) {
    int b, cc;
    cand_decode(cm, n, b, cc);
    int tau = cm.t[b] - cm.koff - cc;
    tau = max(0, min(Tsteps - 1, tau));
    ft = film_time + (size_t)tau * F + foff;
    fo = film_obs + (size_t)item_of(cm.item, b) * F + foff;
  }
  for (int i = threadIdx.x; i < cnt; i += blockDim.x) {
    const int l = i / Cg, c = grp * Cg + (i % Cg);
    float v = (y_at(((size_t)n * Lp + l) * C + c) - mean) * rstd * gam[c] + bet[c];
    v = mish_f(v);
    if (ft) v = (ft[c] + fo[c]) * v + (ft[C + c] + fo[C + c]);
    const size_t prow = (size_t)n * Lp + l + 2;
    if (res_t) v += to_f(res_t[prow * res_pitch + c]);
    if (res_f) v += res_f[prow * C + c];
    dst[prow * dst_pitch + coff + c] = from_f<T>(v);
  }
}

// 2:1 mean pooling along the sequence: dst[n, l + 2, c] = (src[n, 2l + 2, soff + c] + src[n, 2l + 3, soff + c]) / 2.
template <typename T>
__global__ void unet_pool_kernel(const T* __restrict__ src, int src_pitch, int soff, T* __restrict__ dst, int n_cand,
                                 int L_dst, int C, LiveRows lv) {
  pdl_trigger();
  pdl_wait();
  n_cand = live_rows(lv, n_cand);
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (long long)n_cand * L_dst * C) return;
  const int c = (int)(idx % C), l = (int)((idx / C) % L_dst), n = (int)(idx / ((long long)C * L_dst));
  const size_t s0 = ((size_t)n * (2 * L_dst + 4) + 2 * l + 2) * src_pitch + soff + c;
  dst[((size_t)n * (L_dst + 4) + l + 2) * C + c] = from_f<T>(0.5f * (to_f(src[s0]) + to_f(src[s0 + src_pitch])));
}

// 2x repetition along the sequence into channels [0, C) of a wider tensor: dst[n, l + 2, c] = src[n, l/2 + 2, c].
template <typename T>
__global__ void unet_upsample_kernel(const T* __restrict__ src, T* __restrict__ dst, int dst_pitch, int n_cand, int L_dst,
                                     int C, LiveRows lv) {
  pdl_trigger();
  pdl_wait();
  n_cand = live_rows(lv, n_cand);
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (long long)n_cand * L_dst * C) return;
  const int c = (int)(idx % C), l = (int)((idx / C) % L_dst), n = (int)(idx / ((long long)C * L_dst));
  dst[((size_t)n * (L_dst + 4) + l + 2) * dst_pitch + c] = src[((size_t)n * (L_dst / 2 + 4) + l / 2 + 2) * C + c];
}

// Output projection: eps[n, l, :] = X[n, l + 2, :] W_out + b_out; one warp per position; W_outT [A, C] fp32.
template <typename T>
__global__ void unet_head_kernel(const T* __restrict__ X, const float* __restrict__ W_outT, const float* __restrict__ b_out,
                                 CandMap cm, int M, int H, int A, int C) {
  pdl_trigger();
  pdl_wait();
  const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (row >= M) return;
  const int n = row / H, l = row % H;
  if (n >= cand_count(cm, M / H)) return;
  int b, c;
  cand_decode(cm, n, b, c);
  const T* x = X + ((size_t)n * (H + 4) + l + 2) * C;
  float* o = cm.eout + b * cm.e_stride_b + (long long)c * H * A + (long long)l * A;
  for (int a = 0; a < A; ++a) {
    float acc = 0.f;
    for (int i = lane; i < C; i += 32) acc += to_f(x[i]) * W_outT[(size_t)a * C + i];
    acc = warp_sum(acc);
    if (lane == 0) o[a] = acc + b_out[a];
  }
}

}  // namespace tsdp
