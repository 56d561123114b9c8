// End of one draft step of the layer-by-layer transformer drafter, one warp per token row (slot b, token l):
//   eps^ = LN_f(h) W_out + b_out                                  (the drafter's output head)
//   tau = t[b] - k + 1;  mu^_k = posterior mean of (x~_{k-1}, eps^);  x~_k = mu^_k + sigma_tau xi_tau   (Eq. (3), Sec. 3.2)
//   if another draft step follows: h = x~_k W_in + b_in + pos, a = LN1(h)    (the next forward's first two kernels)
// Lane a < A owns action dimension a of its token; the arithmetic is that of head_kernel, draft_step_kernel
// and embed_ln_kernel (shared device functions), so the fused and the separate kernels give the same bits.
// Slots whose drafting is over (k beyond their window) copy the previous latent, as draft_step_kernel does.
#pragma once
#include "common.cuh"
#include "net_kernels.cuh"

namespace tsdp {

template <typename T, int VEC>
__global__ void draft_tail_kernel(float* __restrict__ h, const float* __restrict__ lnf_g, const float* __restrict__ lnf_b,
                                  const float* __restrict__ W_outT, const float* __restrict__ b_out, DdpmTables S,
                                  float* __restrict__ xt, long long xs_b, float* __restrict__ muhat, long long ms_b,
                                  float* __restrict__ eps_d, const int* __restrict__ t, int k, int K, int Tsteps,
                                  const uint64_t* __restrict__ seedp, const EnvParams* __restrict__ envp,
                                  const int* __restrict__ item, const float* __restrict__ W_in, const float* __restrict__ b_in,
                                  const float* __restrict__ pos, const float* __restrict__ ln1_g, const float* __restrict__ ln1_b,
                                  T* __restrict__ a_out, int embed_next, int M, int H, int A,
                                  const int* __restrict__ order, const int* __restrict__ n_live) {
  pdl_trigger();
  pdl_wait();
  constexpr int d = VEC * 128;
  const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (row >= M) return;
  // rows n*H .. n*H+H-1 of the drafter's activations belong to slot b = n, or, when the drafter runs on the
  // round's compacted slot order, to slot order[n] >> 6 (only the first *n_live entries are drafting at step k)
  const int n = row / H, l = row % H;
  if (n_live != nullptr && n >= *n_live) return;
  const int b = order != nullptr ? (order[n] >> 6) : n;
  const int D = H * A;
  float4 v[VEC];
  head_ln_row<VEC>(h + (size_t)row * d, lnf_g, lnf_b, v, lane);
  float e_mine = 0.f;
  for (int a = 0; a < A; ++a) {
    const float e = head_out<VEC>(v, W_outT + (size_t)a * d, b_out[a], lane);
    if (lane == a) e_mine = e;
  }
  const uint64_t seed = *seedp;
  const int tb = t[b];
  const int tau = tb - k + 1;
  const int env = item_of(item, b);
  const bool valid = (tb >= 0) && (tau >= 1) && (k <= env_draft_cap(envp, env, tb, K, Tsteps));
  float xn = 0.f;
  if (lane < A) {
    const int i = l * A + lane;
    const float x = xt[b * xs_b + (long long)(k - 1) * D + i];
    float m = x;
    xn = x;
    if (valid) {
      float z[4];
      normal4(seed, (uint32_t)env, STREAM_XI, (uint32_t)tau, (uint32_t)(i >> 2), z);
      m = posterior_mean(S, x, e_mine, tau);
      xn = ddpm_sample(m, S.sigma[tau], z[i & 3]);
    }
    muhat[b * ms_b + (long long)(k - 1) * D + i] = m;
    xt[b * xs_b + (long long)k * D + i] = xn;
    eps_d[(long long)b * D + i] = e_mine;
  }
  if (embed_next)
    embed_ln_row<T, VEC>([&](int a) { return __shfl_sync(0xffffffffu, xn, a); }, A, W_in, b_in, pos + (size_t)l * d,
                         h + (size_t)row * d, ln1_g, ln1_b, a_out + (size_t)row * d, lane);
}

}  // namespace tsdp
