// Network kernels other than the tensor-core GEMM: the fp32 check-mode GEMM, token embedding,
// LayerNorm, the two small attentions, the output head, the toy MLP and the closed-form Gaussian
// denoiser.  T is the activation type: float in the fp32 check mode, bf16 in the production mode.
#pragma once
#include "common.cuh"
#include "gemm_tcgen05.cuh"

namespace tsdp {

// ------------------------------------------------------------------------------------------------
// fp32 check-mode GEMM (CUDA cores): C[M,N] = A[M,K] W[N,K]^T, same epilogues as the tensor-core one.
// ------------------------------------------------------------------------------------------------
template <int EPI>
__global__ void __launch_bounds__(256)
gemm_simt_kernel(const float* __restrict__ A, const float* __restrict__ W, GemmArgs g) {
  __shared__ float As[16][65], Ws[16][65];
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  const int m0 = blockIdx.y * 64, n0 = blockIdx.x * 64;
  float acc[4][4] = {};
  for (int k0 = 0; k0 < g.K; k0 += 16) {
    for (int i = threadIdx.x; i < 64 * 16; i += 256) {
      const int r = i >> 4, k = i & 15;
      As[k][r] = (m0 + r < g.M) ? A[(size_t)(m0 + r) * g.K + k0 + k] : 0.f;
      Ws[k][r] = (n0 + r < g.N) ? W[(size_t)(n0 + r) * g.K + k0 + k] : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < 16; ++k) {
      float a[4], w[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) { a[i] = As[k][ty * 4 + i]; w[i] = Ws[k][tx * 4 + i]; }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] += a[i] * w[j];
    }
    __syncthreads();
  }
  for (int i = 0; i < 4; ++i) {
    const int row = m0 + ty * 4 + i;
    if (row >= g.M) continue;
    for (int j = 0; j < 4; ++j) {
      const int col = n0 + tx * 4 + j;
      if (col >= g.N) continue;
      float v = acc[i][j] + (g.bias ? g.bias[col] : 0.f);
      if (EPI == EPI_GELU) v = gelu_tanh(v);
      float* o = reinterpret_cast<float*>(g.out) + (size_t)row * g.ldo + col;
      if (EPI == EPI_RESID) v += *o;
      *o = v;
    }
  }
}

// ------------------------------------------------------------------------------------------------
// Token embedding: h[n*H + i, :] = x[n, i, :] W_in + b_in + pos[i, :]      (fp32 residual stream)
// ------------------------------------------------------------------------------------------------
__global__ void embed_kernel(CandMap cm, const float* __restrict__ W_in, const float* __restrict__ b_in,
                             const float* __restrict__ pos, float* __restrict__ h, int H, int A, int d) {
  const int row = blockIdx.x;
  const int n = row / H, i = row % H;
  const int b = n / cm.C, c = n % cm.C;
  const float* x = cm.xin + b * cm.x_stride_b + (long long)c * H * A + (long long)i * A;
  for (int col = threadIdx.x; col < d; col += blockDim.x) {
    float v = b_in[col] + pos[i * d + col];
    for (int a = 0; a < A; ++a) v += x[a] * W_in[a * d + col];
    h[(size_t)row * d + col] = v;
  }
}

// Memory tokens that do not depend on the latent: out[r, :] = in[r, :] W[Din, d] + bias + cpos[row_of(r)].
// Used for the observation tokens (once per chunk) and, with in = the sinusoidal table, at load time.
template <typename T>
__global__ void memtok_kernel(const float* __restrict__ in, int Din, const float* __restrict__ W,
                              const float* __restrict__ bias, const float* __restrict__ cpos, int cpos_mod,
                              int cpos_off, T* __restrict__ out, int d) {
  const int r = blockIdx.x;
  const float* x = in + (size_t)r * Din;
  const float* cp = cpos + (size_t)(cpos_off + (cpos_mod > 0 ? r % cpos_mod : 0)) * d;
  for (int col = threadIdx.x; col < d; col += blockDim.x) {
    float v = cp[col];
    if (W) {
      v += bias[col];
      for (int i = 0; i < Din; ++i) v += x[i] * W[(size_t)i * d + col];
    } else {
      v += x[col];          // identity "projection": Din == d
    }
    out[(size_t)r * d + col] = from_f<T>(v);
  }
}

// ------------------------------------------------------------------------------------------------
// LayerNorm over d (multiple of 128), one warp per row, fp32 in, T out.
// ------------------------------------------------------------------------------------------------
template <typename T, int VEC>
__global__ void ln_kernel(const float* __restrict__ h, const float* __restrict__ gam, const float* __restrict__ bet,
                          T* __restrict__ out, int M) {
  constexpr int d = VEC * 128;
  const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (row >= M) return;
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
#pragma unroll
  for (int j = 0; j < VEC; ++j) {
    const int c = (j * 32 + lane) * 4;
    const float4 gg = reinterpret_cast<const float4*>(gam)[j * 32 + lane];
    const float4 bb = reinterpret_cast<const float4*>(bet)[j * 32 + lane];
    T* o = out + (size_t)row * d + c;
    o[0] = from_f<T>(v[j].x * rstd * gg.x + bb.x);
    o[1] = from_f<T>(v[j].y * rstd * gg.y + bb.y);
    o[2] = from_f<T>(v[j].z * rstd * gg.z + bb.z);
    o[3] = from_f<T>(v[j].w * rstd * gg.w + bb.w);
  }
}

// ------------------------------------------------------------------------------------------------
// Causal self-attention over the H action tokens of one candidate; one warp per (candidate, head).
// qkv [M, 3d] -> out [M, d].  H <= 64, dh = d / heads a multiple of 32 and <= 128.
// ------------------------------------------------------------------------------------------------
template <typename T>
__global__ void self_attn_kernel(const T* __restrict__ qkv, T* __restrict__ out, int n_cand, int H, int d,
                                 int heads) {
  extern __shared__ float sm[];
  const int dh = d / heads;
  const int wpb = blockDim.x >> 5;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int gid = blockIdx.x * wpb + warp;
  if (gid >= n_cand * heads) return;
  const int n = gid / heads, hd = gid % heads;
  float* Q = sm + (size_t)warp * (H * dh + 2 * H * (dh + 1));
  float* Kt = Q + H * dh;
  float* V = Kt + H * (dh + 1);
  const T* base = qkv + (size_t)n * H * 3 * d + hd * dh;
  for (int i = lane; i < H * dh; i += 32) {
    const int r = i / dh, c = i % dh;
    const T* p = base + (size_t)r * 3 * d + c;
    Q[r * dh + c] = to_f(p[0]);
    Kt[r * (dh + 1) + c] = to_f(p[d]);
    V[r * (dh + 1) + c] = to_f(p[2 * d]);
  }
  __syncwarp();
  const float scale = rsqrtf((float)dh);
  for (int r = 0; r < H; ++r) {
    float s0 = -INFINITY, s1 = -INFINITY;
    if (lane <= r) {
      float a = 0.f;
      for (int i = 0; i < dh; ++i) a += Q[r * dh + i] * Kt[lane * (dh + 1) + i];
      s0 = a * scale;
    }
    if (lane + 32 <= r) {
      float a = 0.f;
      for (int i = 0; i < dh; ++i) a += Q[r * dh + i] * Kt[(lane + 32) * (dh + 1) + i];
      s1 = a * scale;
    }
    const float m = warp_max(fmaxf(s0, s1));
    const float p0 = (lane <= r) ? __expf(s0 - m) : 0.f;
    const float p1 = (lane + 32 <= r) ? __expf(s1 - m) : 0.f;
    const float inv = 1.0f / warp_sum(p0 + p1);
    for (int c0 = 0; c0 < dh; c0 += 32) {
      float o = 0.f;
      for (int c = 0; c <= r; ++c) {
        const float p = __shfl_sync(0xffffffffu, c < 32 ? p0 : p1, c & 31);
        o += p * V[c * (dh + 1) + c0 + lane];
      }
      out[((size_t)n * H + r) * d + hd * dh + c0 + lane] = from_f<T>(o * inv);
    }
  }
}

// ------------------------------------------------------------------------------------------------
// Cross-attention to the memory [time token(tau) | obs tokens]; one warp per token row.
// Keys/values are precomputed: kv_time [T, L*2d] (a function of tau only, built at weight load) and
// kv_obs [B*To, L*2d] (built once per chunk); layer l occupies columns [l*2d, (l+1)*2d) = [K | V].
// ------------------------------------------------------------------------------------------------
template <typename T>
__global__ void cross_attn_kernel(const T* __restrict__ q, T* __restrict__ out, const float* __restrict__ kv_time,
                                  const float* __restrict__ kv_obs, CandMap cm, int M, int H, int d, int heads,
                                  int To, int layer, int L, int Tsteps) {
  const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (row >= M) return;
  const int n = row / H;
  const int b = n / cm.C, c = n % cm.C;
  int tau = cm.t[b] - cm.koff - c;
  tau = max(0, min(Tsteps - 1, tau));
  const int dh = d / heads;
  const size_t ld = (size_t)L * 2 * d;
  const float* kt = kv_time + (size_t)tau * ld + (size_t)layer * 2 * d;
  const float* ko = kv_obs + (size_t)b * To * ld + (size_t)layer * 2 * d;
  const float scale = rsqrtf((float)dh);
  const int NK = 1 + To;
  for (int hd = 0; hd < heads; ++hd) {
    float sc[9];
    float m = -INFINITY;
    for (int kx = 0; kx < NK; ++kx) {
      const float* kp = (kx == 0 ? kt : ko + (size_t)(kx - 1) * ld) + hd * dh;
      float a = 0.f;
      for (int i = lane; i < dh; i += 32) a += to_f(q[(size_t)row * d + hd * dh + i]) * kp[i];
      sc[kx] = warp_sum(a) * scale;
      m = fmaxf(m, sc[kx]);
    }
    float l = 0.f;
    for (int kx = 0; kx < NK; ++kx) { sc[kx] = __expf(sc[kx] - m); l += sc[kx]; }
    const float inv = 1.0f / l;
    for (int i = lane; i < dh; i += 32) {
      float o = 0.f;
      for (int kx = 0; kx < NK; ++kx) {
        const float* vp = (kx == 0 ? kt : ko + (size_t)(kx - 1) * ld) + d + hd * dh;
        o += sc[kx] * vp[i];
      }
      out[(size_t)row * d + hd * dh + i] = from_f<T>(o * inv);
    }
  }
}

// ------------------------------------------------------------------------------------------------
// Output head: eps[n, i, :] = LN_f(h[row]) W_out + b_out, one warp per row; W_outT is [A, d] fp32.
// ------------------------------------------------------------------------------------------------
template <int VEC>
__global__ void head_kernel(const float* __restrict__ h, const float* __restrict__ gam, const float* __restrict__ bet,
                            const float* __restrict__ W_outT, const float* __restrict__ b_out, CandMap cm, int M,
                            int H, int A) {
  constexpr int d = VEC * 128;
  const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (row >= M) return;
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
#pragma unroll
  for (int j = 0; j < VEC; ++j) {
    const float4 gg = reinterpret_cast<const float4*>(gam)[j * 32 + lane];
    const float4 bb = reinterpret_cast<const float4*>(bet)[j * 32 + lane];
    v[j].x = v[j].x * rstd * gg.x + bb.x; v[j].y = v[j].y * rstd * gg.y + bb.y;
    v[j].z = v[j].z * rstd * gg.z + bb.z; v[j].w = v[j].w * rstd * gg.w + bb.w;
  }
  const int n = row / H, i = row % H;
  const int b = n / cm.C, c = n % cm.C;
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
// Toy MLP denoiser (fp32): input [latent | sinusoidal(tau) | obs], SiLU hidden layers, linear head.
// One block per candidate; weights [in, out] so that a warp reads a weight row coalesced.
// ------------------------------------------------------------------------------------------------
constexpr int MLP_MAX_LAYERS = 8;
struct MlpWeights {
  int n_lin;                 // hidden layers + 1
  int dims[MLP_MAX_LAYERS + 2];
  const float* W[MLP_MAX_LAYERS + 1];
  const float* b[MLP_MAX_LAYERS + 1];
  int temb;
  const float* temb_table;   // [T, temb]
};

__global__ void mlp_forward_kernel(MlpWeights w, CandMap cm, const float* __restrict__ obs, int obs_len, int D,
                                   int Tsteps) {
  extern __shared__ float sm[];
  const int n = blockIdx.x;
  const int b = n / cm.C, c = n % cm.C;
  int tau = cm.t[b] - cm.koff - c;
  tau = max(0, min(Tsteps - 1, tau));
  int maxw = 0;
  for (int l = 0; l <= w.n_lin; ++l) maxw = max(maxw, w.dims[l]);
  float* cur = sm;
  float* nxt = sm + maxw;
  const float* x = cm.xin + b * cm.x_stride_b + (long long)c * D;
  for (int i = threadIdx.x; i < w.dims[0]; i += blockDim.x) {
    float v;
    if (i < D) v = x[i];
    else if (i < D + w.temb) v = w.temb_table[tau * w.temb + (i - D)];
    else v = obs[(size_t)b * obs_len + (i - D - w.temb)];
    cur[i] = v;
  }
  __syncthreads();
  for (int l = 0; l < w.n_lin; ++l) {
    const int nin = w.dims[l], nout = w.dims[l + 1];
    for (int j = threadIdx.x; j < nout; j += blockDim.x) {
      float a = w.b[l][j];
      for (int i = 0; i < nin; ++i) a += cur[i] * w.W[l][(size_t)i * nout + j];
      nxt[j] = (l + 1 < w.n_lin) ? silu(a) : a;
    }
    __syncthreads();
    float* tmp = cur; cur = nxt; nxt = tmp;
  }
  float* o = cm.eout + b * cm.e_stride_b + (long long)c * D;
  for (int i = threadIdx.x; i < D; i += blockDim.x) o[i] = cur[i];
}

// Closed-form denoiser of iid N(m0, s0^2) data: eps = sqrt(1-abar)(x - sqrt(abar) m0)/(abar s0^2 + 1 - abar).
__global__ void gauss_forward_kernel(DdpmTables S, float m0, float s0, CandMap cm, int n_cand, int D) {
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (long long)n_cand * D) return;
  const int n = (int)(idx / D), i = (int)(idx % D);
  const int b = n / cm.C, c = n % cm.C;
  int tau = cm.t[b] - cm.koff - c;
  tau = max(0, min(S.T - 1, tau));
  const float sab = S.sqrt_ab[tau], s1 = S.sqrt_1mab[tau];
  const float ab = sab * sab;
  const float x = cm.xin[b * cm.x_stride_b + (long long)c * D + i];
  cm.eout[b * cm.e_stride_b + (long long)c * D + i] = s1 * (x - sab * m0) / (ab * s0 * s0 + s1 * s1);
}

}  // namespace tsdp
