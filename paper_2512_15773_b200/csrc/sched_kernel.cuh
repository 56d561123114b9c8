// Inference of the speculative-decoding scheduler (Sec. 3.3): three stream encoders (observation, last
// action chunk, task progress), an aggregating MLP, five outputs squashed into the speculative
// parameters of each environment.  A tiny network: one block per environment, one thread per hidden
// unit, weights read through the read-only cache; it runs once per chunk beside the chunk set-up.
#pragma once
#include "common.cuh"

namespace tsdp {

constexpr int SCHED_HID = 64, SCHED_PROG = 16, SCHED_CAT = 2 * SCHED_HID + SCHED_PROG, SCHED_OUT = 5;

struct SchedWeights {            // W [in, out] fp32, as in the weight blob
  const float *W_o, *b_o, *W_a, *b_a, *W_p, *b_p, *W_1, *b_1, *W_2, *b_2;
};

__global__ void __launch_bounds__(128)
sched_mlp_kernel(SchedWeights w, const float* __restrict__ obs, int obs_len, const float* __restrict__ prev_act, int D,
                 const float* __restrict__ progress, int K_max, EnvParams* __restrict__ out, float* __restrict__ params_out) {
  pdl_trigger();
  pdl_wait();
  __shared__ float cat[SCHED_CAT], g[SCHED_HID], y[SCHED_OUT];
  const int b = blockIdx.x, j = threadIdx.x;
  if (j < SCHED_HID) {                              // observation stream
    float a = w.b_o[j];
    for (int i = 0; i < obs_len; ++i) a += obs[(size_t)b * obs_len + i] * __ldg(w.W_o + (size_t)i * SCHED_HID + j);
    cat[j] = tanhf(a);
  } else {                                          // action stream
    const int u = j - SCHED_HID;
    float a = w.b_a[u];
    for (int i = 0; i < D; ++i) a += prev_act[(size_t)b * D + i] * __ldg(w.W_a + (size_t)i * SCHED_HID + u);
    cat[SCHED_HID + u] = tanhf(a);
  }
  if (j < SCHED_PROG) cat[2 * SCHED_HID + j] = tanhf(progress[b] * w.W_p[j] + w.b_p[j]);
  __syncthreads();
  if (j < SCHED_HID) {
    float a = w.b_1[j];
    for (int i = 0; i < SCHED_CAT; ++i) a += cat[i] * __ldg(w.W_1 + (size_t)i * SCHED_HID + j);
    g[j] = tanhf(a);
  }
  __syncthreads();
  if (j < SCHED_OUT) {
    float a = w.b_2[j];
    for (int i = 0; i < SCHED_HID; ++i) a += g[i] * w.W_2[i * SCHED_OUT + j];
    y[j] = 1.0f / (1.0f + expf(-a));                // sigmoid of the raw output
  }
  __syncthreads();
  if (j == 0) {
    EnvParams e;
    e.sigma_scale = 1.0f + 2.0f * y[0];
    e.log_lambda = logf(y[1]);
    for (int s = 0; s < 3; ++s) e.K[s] = 1 + (int)rintf((float)(K_max - 1) * y[2 + s]);
    out[b] = e;
    if (params_out) {
      float* o = params_out + (size_t)b * 8;
      o[0] = e.sigma_scale; o[1] = y[1];
      for (int s = 0; s < 3; ++s) { o[2 + s] = (float)e.K[s]; o[5 + s] = 1.0f + (float)(K_max - 1) * y[2 + s]; }
    }
  }
}

}  // namespace tsdp
