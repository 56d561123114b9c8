// Forward evaluation of the drafter's distillation objective (Sec. 3.2, "Draft model"): the noising of clean
// chunks and the per-sample loss terms.  The two network forwards in between are the ordinary ones.
#pragma once
#include "common.cuh"

namespace tsdp {

// Sample n: t_n = floor(T u_n) with u_n the uniform of (seed, n, timestep code 0); eps_n the INIT-stream
// normals of (seed, n);  x_t = sqrt(abar_t) x0 + sqrt(1 - abar_t) eps  into candidate slot 0 of xt[n].
__global__ void distill_noise_kernel(DdpmTables S, const float* __restrict__ x0, float* __restrict__ xt, long long xs_b,
                                     int* __restrict__ t, int D, const uint64_t* __restrict__ seedp) {
  const uint64_t seed = *seedp;
  const int n = blockIdx.x;
  const int tn = min(S.T - 1, (int)((double)uniform1(seed, (uint32_t)n, 0u) * (double)S.T));
  if (threadIdx.x == 0) t[n] = tn;
  const float a = S.sqrt_ab[tn], b = S.sqrt_1mab[tn];
  const int nq = (D + 3) >> 2;
  for (int q = threadIdx.x; q < nq; q += blockDim.x) {
    float z[4];
    normal4(seed, (uint32_t)n, STREAM_INIT, 0u, (uint32_t)q, z);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int i = 4 * q + j;
      if (i < D) xt[n * xs_b + i] = __fmaf_rn(b, z[j], __fmul_rn(a, x0[(long long)n * D + i]));
    }
  }
}

// out[n] = { |m^ - m|^2,  |(mu^ - mu) / sigma_t|^2 (0 at t = 0),  1 if t >= 1 else 0 } for sample n; m = eps_base,
// m^ = eps_draft are the networks' outputs on x_t.  One block per sample.
__global__ void distill_terms_kernel(DdpmTables S, const float* __restrict__ xt, long long xs_b,
                                     const float* __restrict__ eps_base, long long eb_b, const float* __restrict__ eps_draft,
                                     long long ed_b, const int* __restrict__ t, int D, float* __restrict__ out) {
  __shared__ float red[2][32];
  const int n = blockIdx.x;
  const int tn = t[n];
  const float inv_sigma = tn >= 1 ? 1.0f / S.sigma[tn] : 0.f;
  float sp = 0.f, sn = 0.f;
  for (int i = threadIdx.x; i < D; i += blockDim.x) {
    const float x = xt[n * xs_b + i], m = eps_base[n * eb_b + i], mh = eps_draft[n * ed_b + i];
    const float dm = mh - m;
    sp += dm * dm;
    if (tn >= 1) {
      const float d = (posterior_mean(S, x, mh, tn) - posterior_mean(S, x, m, tn)) * inv_sigma;
      sn += d * d;
    }
  }
  sp = warp_sum(sp); sn = warp_sum(sn);
  if ((threadIdx.x & 31) == 0) { red[0][threadIdx.x >> 5] = sp; red[1][threadIdx.x >> 5] = sn; }
  __syncthreads();
  if (threadIdx.x == 0) {
    float a = 0.f, b = 0.f;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) { a += red[0][w]; b += red[1][w]; }
    out[3 * n] = a; out[3 * n + 1] = b; out[3 * n + 2] = tn >= 1 ? 1.f : 0.f;
  }
}

}  // namespace tsdp
