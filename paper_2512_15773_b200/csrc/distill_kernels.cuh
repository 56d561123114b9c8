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

// ------------------------------------------------------------------------------------------------
// One gradient step of the objective on the closed-form Gaussian drafter (Sec. 3.2, "Draft Model Training":
// the base model is frozen, only the drafter's parameters theta = (m0, s0) move).
//   m^(x, t) = s1 (x - sab m0) / v,   v = abar s0^2 + (1 - abar),   s1 = sqrt(1 - abar), sab = sqrt(abar)
//   d m^/d m0 = -s1 sab / v,          d m^/d s0 = -s1 (x - sab m0) 2 abar s0 / v^2
//   (mu^ - mu)/sigma_t = -c_t (m^ - m),  c_t = c_x0 s1 / (sab sigma_t)      (posterior mean affine in the output)
// Per sample n the first kernel writes { |r|^2, c_t^2 (0 at t = 0), [t >= 1], 2 <r, dm^/dm0>, 2 <r, dm^/ds0> },
// r = m^ - m; the second reduces them in double, forms
//   L_pred = sum |r|^2 / N,  L_norm = sum c^2 |r|^2 / N_1,  dL/dtheta = sum (lambda1/N + lambda2 c^2/N_1) G_theta
// and applies theta <- theta - lr dL/dtheta.
// ------------------------------------------------------------------------------------------------
__global__ void distill_gauss_grad_kernel(DdpmTables S, const float* __restrict__ xt, long long xs_b,
                                          const float* __restrict__ eps_base, long long eb_b, const int* __restrict__ t, int D,
                                          const float* __restrict__ theta, float* __restrict__ out) {
  __shared__ float red[3][32];
  const int n = blockIdx.x;
  const int tn = t[n];
  const float m0 = theta[0], s0 = theta[1];
  const float sab = S.sqrt_ab[tn], s1 = S.sqrt_1mab[tn];
  const float ab = sab * sab;
  const float v = ab * s0 * s0 + s1 * s1;
  const float dm = -s1 * sab / v;
  const float ds_c = -s1 * 2.0f * ab * s0 / (v * v);
  float sr = 0.f, gm = 0.f, gs = 0.f;
  for (int i = threadIdx.x; i < D; i += blockDim.x) {
    const float x = xt[n * xs_b + i];
    const float u = x - sab * m0;
    const float r = s1 * u / v - eps_base[n * eb_b + i];
    sr += r * r; gm += r * dm; gs += r * ds_c * u;
  }
  sr = warp_sum(sr); gm = warp_sum(gm); gs = warp_sum(gs);
  if ((threadIdx.x & 31) == 0) { red[0][threadIdx.x >> 5] = sr; red[1][threadIdx.x >> 5] = gm; red[2][threadIdx.x >> 5] = gs; }
  __syncthreads();
  if (threadIdx.x == 0) {
    float a = 0.f, b = 0.f, c = 0.f;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) { a += red[0][w]; b += red[1][w]; c += red[2][w]; }
    float c2 = 0.f;
    if (tn >= 1) { const float ct = S.c_x0[tn] * s1 / (sab * S.sigma[tn]); c2 = ct * ct; }
    out[5 * n] = a; out[5 * n + 1] = c2; out[5 * n + 2] = tn >= 1 ? 1.f : 0.f; out[5 * n + 3] = 2.f * b; out[5 * n + 4] = 2.f * c;
  }
}

// res[7] = { L_pred, L_norm, L (before the step), dL/dm0, dL/ds0, m0', s0' }; theta is updated in place.
__global__ void distill_gauss_update_kernel(const float* __restrict__ terms, int N, float lambda1, float lambda2, float lr,
                                            float* __restrict__ theta, double* __restrict__ res) {
  __shared__ double acc[7][256];
  double a[7] = {0, 0, 0, 0, 0, 0, 0};      // sum r2, sum c2 r2, N1, sum Gm, sum Gs, sum c2 Gm, sum c2 Gs
  for (int n = threadIdx.x; n < N; n += blockDim.x) {
    const double r2 = terms[5 * n], c2 = terms[5 * n + 1], fl = terms[5 * n + 2], gm = terms[5 * n + 3], gs = terms[5 * n + 4];
    a[0] += r2; a[1] += c2 * r2; a[2] += fl; a[3] += gm; a[4] += gs; a[5] += c2 * gm; a[6] += c2 * gs;
  }
  for (int j = 0; j < 7; ++j) acc[j][threadIdx.x] = a[j];
  __syncthreads();
  for (int o = blockDim.x >> 1; o > 0; o >>= 1) {
    if ((int)threadIdx.x < o)
      for (int j = 0; j < 7; ++j) acc[j][threadIdx.x] += acc[j][threadIdx.x + o];
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    const double N1 = acc[2][0];
    const double Lp = acc[0][0] / N, Ln = N1 > 0 ? acc[1][0] / N1 : 0.0;
    const double gm = lambda1 * acc[3][0] / N + (N1 > 0 ? lambda2 * acc[5][0] / N1 : 0.0);
    const double gs = lambda1 * acc[4][0] / N + (N1 > 0 ? lambda2 * acc[6][0] / N1 : 0.0);
    const double m1 = (double)theta[0] - (double)lr * gm, s1 = (double)theta[1] - (double)lr * gs;
    theta[0] = (float)m1; theta[1] = (float)s1;
    res[0] = Lp; res[1] = Ln; res[2] = (double)lambda1 * Lp + (double)lambda2 * Ln; res[3] = gm; res[4] = gs;
    res[5] = (double)theta[0]; res[6] = (double)theta[1];
  }
}

}  // namespace tsdp
