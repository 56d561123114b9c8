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

// ---- warp-level tensor-core helpers (mma.sync m16n8k16 bf16, ldmatrix) shared by the attention kernels
__device__ __forceinline__ void mma_bf16_16816(float c[4], const uint32_t a[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 h2 = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&h2);
}

// Four 8x8 b16 matrices from shared memory: lanes 8i..8i+7 give the 16-byte row addresses of matrix i.
// Plain: lane l receives M[l/4][2(l%4) .. +1] -- the B fragment of a [n][k] (K-major) tile.
// Transposed: lane l receives M[2(l%4) .. +1][l/4] -- the B fragment of a [k][n] tile (values V of attention).
__device__ __forceinline__ void ldmatrix_x4(uint32_t r[4], const void* smem_row) {
  const uint32_t a = (uint32_t)__cvta_generic_to_shared(smem_row);
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(a));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t r[4], const void* smem_row) {
  const uint32_t a = (uint32_t)__cvta_generic_to_shared(smem_row);
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(a));
}

// Attention of one (candidate, head) with at most 16 tokens by one warp, operands already in shared memory:
// sQ, sK, sV are [16][DH + 8] bf16 tiles (rows past H zero).  S = Q K^T and O = P V on mma.sync m16n8k16 (Q with
// 4-byte loads, K through ldmatrix, V through ldmatrix.trans), softmax in the accumulator registers.  The
// normalised output tile overwrites sQ.  Used by self_attn_tile_kernel and by the fused QKV epilogue of the
// tensor-core GEMM, which therefore produce the same bits.
template <int DH>
__device__ __forceinline__ void attn16_from_smem(__nv_bfloat16* sQ, const __nv_bfloat16* sK, const __nv_bfloat16* sV, int H,
                                                 int causal, int lane) {
  constexpr int KS = DH / 16, NO = DH / 8, P = DH + 8;
  const int g = lane >> 2, tg = lane & 3;
  uint32_t qa[KS][4];
#pragma unroll
  for (int ks = 0; ks < KS; ++ks) {
    const __nv_bfloat16* q0 = sQ + g * P + ks * 16 + 2 * tg;
    qa[ks][0] = *reinterpret_cast<const uint32_t*>(q0);
    qa[ks][1] = *reinterpret_cast<const uint32_t*>(q0 + 8 * P);
    qa[ks][2] = *reinterpret_cast<const uint32_t*>(q0 + 8);
    qa[ks][3] = *reinterpret_cast<const uint32_t*>(q0 + 8 * P + 8);
  }
  const int nkt = causal ? 2 : (H + 7) >> 3;
  float s[2][4];
#pragma unroll
  for (int nt = 0; nt < 2; ++nt) {
    s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f;
    if (nt < nkt) {
#pragma unroll
      for (int ks = 0; ks < KS; ks += 2) {
        uint32_t b[4];
        ldmatrix_x4(b, sK + (nt * 8 + (lane & 7)) * P + ks * 16 + 8 * (lane >> 3));
        mma_bf16_16816(s[nt], qa[ks], b[0], b[1]);
        mma_bf16_16816(s[nt], qa[ks + 1], b[2], b[3]);
      }
    }
  }
  const float scale = rsqrtf((float)DH);
  const int r0 = g, r1 = g + 8;
  float m0 = -INFINITY, m1 = -INFINITY;
#pragma unroll
  for (int nt = 0; nt < 2; ++nt) {
    if (nt < nkt) {
      const int col = nt * 8 + 2 * tg;
      const int lim0 = causal ? r0 : H, lim1 = causal ? r1 : H;
      s[nt][0] = (col <= lim0 && col < H) ? s[nt][0] * scale : -INFINITY;
      s[nt][1] = (col + 1 <= lim0 && col + 1 < H) ? s[nt][1] * scale : -INFINITY;
      s[nt][2] = (col <= lim1 && col < H) ? s[nt][2] * scale : -INFINITY;
      s[nt][3] = (col + 1 <= lim1 && col + 1 < H) ? s[nt][3] * scale : -INFINITY;
      m0 = fmaxf(m0, fmaxf(s[nt][0], s[nt][1]));
      m1 = fmaxf(m1, fmaxf(s[nt][2], s[nt][3]));
    }
  }
  m0 = fmaxf(m0, __shfl_xor_sync(0xffffffffu, m0, 1)); m0 = fmaxf(m0, __shfl_xor_sync(0xffffffffu, m0, 2));
  m1 = fmaxf(m1, __shfl_xor_sync(0xffffffffu, m1, 1)); m1 = fmaxf(m1, __shfl_xor_sync(0xffffffffu, m1, 2));
  // rows beyond H have no visible key: keep the arithmetic finite, their output is never stored
  if (m0 == -INFINITY) m0 = 0.f;
  if (m1 == -INFINITY) m1 = 0.f;
  float l0 = 0.f, l1 = 0.f;
#pragma unroll
  for (int nt = 0; nt < 2; ++nt) {
    if (nt < nkt) {
      s[nt][0] = __expf(s[nt][0] - m0); s[nt][1] = __expf(s[nt][1] - m0);
      s[nt][2] = __expf(s[nt][2] - m1); s[nt][3] = __expf(s[nt][3] - m1);
      l0 += s[nt][0] + s[nt][1]; l1 += s[nt][2] + s[nt][3];
    }
  }
  l0 += __shfl_xor_sync(0xffffffffu, l0, 1); l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
  l1 += __shfl_xor_sync(0xffffffffu, l1, 1); l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
  const float inv0 = l0 > 0.f ? 1.0f / l0 : 0.f, inv1 = l1 > 0.f ? 1.0f / l1 : 0.f;
  uint32_t pa[4];
  pa[0] = pack_bf16(s[0][0], s[0][1]); pa[1] = pack_bf16(s[0][2], s[0][3]);
  pa[2] = pack_bf16(s[1][0], s[1][1]); pa[3] = pack_bf16(s[1][2], s[1][3]);
  __syncwarp();                                   // every lane has its Q fragments: the Q rows become the output tile
#pragma unroll
  for (int no = 0; no < NO; no += 2) {
    float o0[4] = {0.f, 0.f, 0.f, 0.f}, o1[4] = {0.f, 0.f, 0.f, 0.f};
    uint32_t b[4];
    ldmatrix_x4_trans(b, sV + ((lane & 7) + 8 * ((lane >> 3) & 1)) * P + no * 8 + 8 * (lane >> 4));
    mma_bf16_16816(o0, pa, b[0], b[1]);
    mma_bf16_16816(o1, pa, b[2], b[3]);
    const int col = no * 8 + 2 * tg;
    *reinterpret_cast<uint32_t*>(sQ + g * P + col) = pack_bf16(o0[0] * inv0, o0[1] * inv0);
    *reinterpret_cast<uint32_t*>(sQ + (g + 8) * P + col) = pack_bf16(o0[2] * inv1, o0[3] * inv1);
    *reinterpret_cast<uint32_t*>(sQ + g * P + col + 8) = pack_bf16(o1[0] * inv0, o1[1] * inv0);
    *reinterpret_cast<uint32_t*>(sQ + (g + 8) * P + col + 8) = pack_bf16(o1[2] * inv1, o1[3] * inv1);
  }
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
