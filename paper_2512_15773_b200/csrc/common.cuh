// Shared device helpers of the TS-DP CUDA path: Philox4x32-10 noise streams, the DDPM posterior,
// warp reductions.  Written for sm_100a; nothing here is shared with the CPU oracle.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace tsdp {

// ----------------------------------------------------------------------------------------------
// Counter-based noise.  Every random number is a pure function of (seed, env, stream, timestep,
// element): counter = (quad index, timestep code, env, stream), key = seed.  A draft at timestep
// tau and a base step at tau therefore see the same xi_tau, which makes "drafter == base"
// reproduce vanilla DDPM bit for bit (Sec. 3.2: the rollout retains its noise realisations).
// ----------------------------------------------------------------------------------------------
enum : uint32_t { STREAM_INIT = 0, STREAM_XI = 1, STREAM_U = 2 };

__device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                               uint32_t k0, uint32_t k1, uint32_t out[4]) {
  const uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u, W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint32_t hi0 = __umulhi(M0, c0), lo0 = M0 * c0;
    const uint32_t hi1 = __umulhi(M1, c2), lo1 = M1 * c2;
    const uint32_t n0 = hi1 ^ c1 ^ k0, n2 = hi0 ^ c3 ^ k1;
    c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
    k0 += W0; k1 += W1;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// ((n >> 9) + 0.5) * 2^-23: in (0,1), exact in fp32.
__device__ __forceinline__ float bits_to_unit(uint32_t n) {
  return (__uint2float_rn(n >> 9) + 0.5f) * 1.1920928955078125e-07f;
}

// Four standard normals of counter quad `quad`: lanes (0,1) and (2,3) are the cosine / sine branches
// of one Box-Muller pair each.
__device__ __forceinline__ void normal4(uint64_t seed, uint32_t env, uint32_t stream, uint32_t tcode,
                                        uint32_t quad, float z[4]) {
  uint32_t w[4];
  philox4x32_10(quad, tcode, env, stream, (uint32_t)seed, (uint32_t)(seed >> 32), w);
#pragma unroll
  for (int p = 0; p < 2; ++p) {
    const float r = sqrtf(-2.0f * logf(bits_to_unit(w[2 * p])));
    float s, c;
    sincospif(2.0f * bits_to_unit(w[2 * p + 1]), &s, &c);
    z[2 * p] = r * c;
    z[2 * p + 1] = r * s;
  }
}

__device__ __forceinline__ float uniform1(uint64_t seed, uint32_t env, uint32_t tau) {
  uint32_t w[4];
  philox4x32_10(0u, tau, env, STREAM_U, (uint32_t)seed, (uint32_t)(seed >> 32), w);
  return bits_to_unit(w[0]);
}

// ----------------------------------------------------------------------------------------------
// DDPM scheduler S (the paper's x_{t-1} = S(m_t, t, x_t), Sec. 3.2): per-timestep coefficients of
// the Gaussian reverse transition, tabulated once per context in fp64 and stored as fp32.
// ----------------------------------------------------------------------------------------------
struct DdpmTables {
  const float* sqrt_ab;     // sqrt(abar_t)
  const float* sqrt_1mab;   // sqrt(1 - abar_t)
  const float* c_x0;        // sqrt(abar_{t-1}) beta_t / (1 - abar_t)
  const float* c_xt;        // sqrt(alpha_t) (1 - abar_{t-1}) / (1 - abar_t)
  const float* sigma;       // sqrt(beta_t (1 - abar_{t-1}) / (1 - abar_t)), sigma_0 = 0
  int T;
  float clip;               // clamp x0_hat to +-clip when > 0
};

// The operations are spelled out (fused multiply-adds and roundings fixed) so that every kernel that takes a
// reverse step -- draft step, acceptance kernel, cluster kernel -- rounds identically: with drafter == base the
// speculative chunk then equals vanilla DDPM bit for bit.
__device__ __forceinline__ float posterior_mean(const DdpmTables& S, float x, float eps, int tau) {
  float x0 = __fdiv_rn(__fmaf_rn(-S.sqrt_1mab[tau], eps, x), S.sqrt_ab[tau]);
  if (S.clip > 0.f) x0 = fminf(fmaxf(x0, -S.clip), S.clip);
  return __fmaf_rn(S.c_x0[tau], x0, __fmul_rn(S.c_xt[tau], x));
}
// x_{t-1} = mu + sigma xi
__device__ __forceinline__ float ddpm_sample(float mu, float sigma, float xi) { return __fmaf_rn(sigma, xi, mu); }

// Programmatic dependent launch: a kernel signals early that its successor in the stream may be
// scheduled, and waits (after whatever set-up touches no shared data) until every kernel it depends on
// has completed and its memory is visible.  Both are no-ops for a kernel launched without the attribute.
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

__device__ __forceinline__ float to_f(float v) { return v; }
__device__ __forceinline__ float to_f(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

__device__ __forceinline__ float gelu_tanh(float v) {
  const float k = 0.7978845608028654f;   // sqrt(2/pi)
  return 0.5f * v * (1.0f + tanhf(k * (v + 0.044715f * v * v * v)));
}
__device__ __forceinline__ float silu(float v) { return v / (1.0f + __expf(-v)); }

// Which candidate rows a forward pass covers.  Dense form (list == null): candidate n = (env b = n / C, slot
// c = n % C).  Compacted form: candidate n = (b, c) = (list[n] >> 6, list[n] & 63), and only the first *n_live
// entries exist -- the round's plan (round_plan_kernel) lists the candidates that are still needed, so that finished
// environments and draft slots beyond an environment's window cost nothing.  Either way the candidate reads its
// latent at xin + b*x_stride_b + c*D, is evaluated at timestep clamp(t[b] - koff - c, 0, T-1) and writes eps at
// eout + b*e_stride_b + c*D.  b is a slot of the batch; which request (environment-chunk) the slot is working on
// is item[b].
struct CandMap {
  const float* xin;  long long x_stride_b;
  float* eout;       long long e_stride_b;
  const int* t;      int C;  int koff;
  const int* item;   // slot b currently serves request item[b] (its observation, its noise streams); null: b
  const int* list;   // compacted candidate list (null: dense)
  const int* n_live; // number of entries of `list` in use (device word written earlier in the stream)
};
__device__ __forceinline__ int item_of(const int* item, int b) { return item ? item[b] : b; }
__device__ __forceinline__ void cand_decode(const CandMap& cm, int n, int& b, int& c) {
  if (cm.list) { const int v = cm.list[n]; b = v >> 6; c = v & 63; }
  else { b = n / cm.C; c = n % cm.C; }
}
// Candidates this pass really has (n_static is what the launch was sized for).
__device__ __forceinline__ int cand_count(const CandMap& cm, int n_static) {
  return cm.n_live ? min(*cm.n_live, n_static) : n_static;
}
// The same for kernels that only see rows: rows = *n * mul + add, never more than the launch was sized for.
struct LiveRows {
  const int* n;  int mul;  int add;
};
__device__ __forceinline__ int live_rows(const LiveRows& lv, int rows_static) {
  if (lv.n == nullptr) return rows_static;
  const int v = *lv.n * lv.mul + lv.add;
  return v < 0 ? 0 : (v < rows_static ? v : rows_static);
}

// Per-round speculative parameters (the scheduler's action space, Sec. 3.3: draft steps, acceptance
// threshold, sigma scale).
struct RoundParams {
  int K;
  int mode;           // 0: U <= min(1, alpha)   1: min(1, alpha) >= lambda
  float log_lambda;
  float sigma_scale;
  int bonus;
};

// Per-environment speculative parameters written by the scheduler network (Sec. 3.3: sigma scale,
// acceptance threshold, draft steps for the early / middle / late denoising stage).
struct EnvParams {
  float sigma_scale;
  float log_lambda;
  int K[3];
};

// Denoising stage of timestep t: 0 early (t >= 4T/5), 2 late (t < T/5), 1 in between.
__device__ __forceinline__ int stage_of(int t, int T) { return t >= (4 * T) / 5 ? 0 : (t < T / 5 ? 2 : 1); }

// Draft steps environment b may take in this round: the round's K, capped by the scheduler's choice.
__device__ __forceinline__ int env_draft_cap(const EnvParams* envp, int env, int tb, int K, int T) {
  if (envp == nullptr || tb < 0) return K;
  const int kb = envp[env].K[stage_of(tb, T)];
  return kb < K ? kb : K;
}

// Device-side counters behind tsdp_stats.
struct DevStats {
  unsigned long long env_rounds, base_evals, draft_evals, drafts_tested, drafts_accepted, rejections,
      bonus_steps, steps_advanced, chunks_done, draft_rounds, cand_computed, draft_computed;
  unsigned long long hist_drafted[1024], hist_tested[1024], hist_accepted[1024];
};

}  // namespace tsdp
