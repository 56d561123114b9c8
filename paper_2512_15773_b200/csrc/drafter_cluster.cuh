// Persistent drafter: the whole K-step draft rollout of one environment (Sec. 3.2 "Draft Generation
// Procedure", Eq. (3)) in ONE kernel launch, for small batches where the rollout is latency-bound.
//
// One thread-block cluster of DC_CS CTAs serves one environment at a time.  Every CTA owns a 1/DC_CS
// slice (a block of output columns) of every weight matrix of the drafter -- kept in shared memory
// for the whole launch when it fits beside the activations, otherwise read in place through the L2 --
// and a full replica of the activations of the 16-token sequence.  A linear layer
// is computed as Y[:, slice] = X W_slice^T on mma.sync m16n8k16 (the sequence is one 16-row tile),
// and each CTA writes its slice of Y into the replicas of all CTAs through distributed shared
// memory (4 such exchanges per block: qkv, attention projection, MLP up, MLP down; 6 when the
// cross-attention is not folded into the memory tokens).  LayerNorm, the attentions, the folded
// cross-attention products, the head, the DDPM posterior and the noise are cheap enough to be
// recomputed by every CTA, which saves their broadcasts.  Reductions are warp shuffles.
// A stage's slices travel as 16-byte st.async stores that also count their bytes on an mbarrier of the receiving
// CTA; a CTA goes on as soon as the bytes of all eight slices have arrived (a bounded mbarrier wait), with no
// release fence and no cluster-wide barrier per stage.  Two mbarriers alternate between consecutive stages: a CTA
// can run at most one stage ahead of the slowest one (it needs everybody's slice of the previous stage), so the
// bytes of stage s + 1 never land on the barrier that still counts stage s.  The same reasoning covers the
// buffers: what a fast CTA writes remotely in stage s + 1 is never what a slower one still reads in stage s.
// (TSDP_NO_ASYNC_BCAST selects plain distributed-shared-memory stores and barrier.cluster instead.)
// All CTAs of a cluster make the same sequence of stages because the control flow depends only on (t[b], k).
#pragma once
#include <cooperative_groups.h>
#include "common.cuh"
#include "gemm_tcgen05.cuh"
#include "net_kernels.cuh"

namespace tsdp {
namespace cg = cooperative_groups;

constexpr int DC_CS = 8;          // CTAs per cluster (the portable maximum)
constexpr int DC_THREADS = 256;
constexpr int DC_WARPS = DC_THREADS / 32;
constexpr int DC_ROWS = 16;       // one m16 tile: H <= 16
constexpr int DC_MAX_LAYERS = 8;
constexpr int DC_MAX_NK = 4;      // memory tokens: time token + at most 3 observation tokens
constexpr int DC_PU = 40;         // folded cross-attention: row pitch (bf16) of the [.. x 32] operands of its second product

__device__ __forceinline__ uint32_t dc_mapa(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void dc_st_async16(uint32_t remote, const uint4& v, uint32_t remote_bar) {
  asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v4.b32 [%0], {%1,%2,%3,%4}, [%5];"
               ::"r"(remote), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w), "r"(remote_bar) : "memory");
}
__device__ __forceinline__ void dc_st_cluster16(uint32_t remote, const uint4& v) {
  asm volatile("st.shared::cluster.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(remote), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

template <int BYTES>
__device__ __forceinline__ void dc_cp_async(void* smem_dst, const void* gsrc) {
  const uint32_t dst = (uint32_t)__cvta_generic_to_shared(smem_dst);
  if (BYTES == 16) asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(gsrc) : "memory");
  else asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(dst), "l"(gsrc) : "memory");
}

struct DcLayer {
  const __nv_bfloat16 *Wqkv, *Wo, *Wq2, *Wo2, *W1, *W2;      // [out, in] bf16
  const float *bqkv, *bo, *bq2, *bo2, *b1, *b2;
  const float *ln1_g, *ln1_b, *ln2_g, *ln2_b, *ln3_g, *ln3_b;
};

struct DcParams {
  DcLayer L[DC_MAX_LAYERS];
  int layers, heads, H, A, To, T;
  const float *W_in, *b_in, *pos;                            // [A, d], [d], [H, d]
  const float *lnf_g, *lnf_b, *W_outT, *b_out;               // W_outT [A, d]
  const float *kv_time, *kv_obs;                             // [T, L*2d], [B*To, L*2d]
  // cross-attention folded into the memory tokens (xattn_fold.cuh): per-token tables kq [L][heads][d],
  // ut [L][heads/2][d][2] (bf16) and c [L][heads] (fp32); fold = 0 runs the projections and the attention instead
  const __nv_bfloat16 *kq_time, *ut_time, *kq_obs, *ut_obs;
  const float *c_time, *c_obs;
  int fold;
  int async_bcast;                                           // 1: slices travel by st.async and are counted by the receivers' mbarriers
  int* status;                                               // set to 5 if a wait gives up
  DdpmTables S;
  float* xt; long long xs_b;                                 // candidates [B, Kmax+1, D]
  float* muhat; long long ms_b;                              // drafter means [B, Kmax, D]
  const int* t;
  const uint64_t* seed;
  int resident;                                              // 1: weight slices live in shared memory for the whole launch
  // mode 0: draft rollout (K steps per slot, writes xt / muhat).  mode 1: verification -- one forward per
  // (slot, candidate c < C) at timestep t[slot] - c, reading xt[slot, c] and writing eps[slot, c].
  int mode, C;
  float* eps; long long es_b;
  const EnvParams* envp;                                     // per-request draft cap, or null
  const int* item;                                           // slot -> request it serves, or null
  int B, K;
};

// Shared-memory plan of one CTA (bytes), for model width d.  Weight rows are padded by 8 elements so
// that fragment loads of 8 consecutive rows fall into different banks.
struct DcSmem {
  int w_layer;      // bytes of one layer's weight slices
  int off_h, off_a, off_qkv, off_q2, off_f, off_red, off_kv, off_x, off_posb, off_win, off_par, total;
};
__host__ __device__ inline DcSmem dc_smem_plan(int d, int layers, int A, bool resident) {
  DcSmem p;
  const int pw = d + 8, pw4 = 4 * d + 8;
  const int rows_d = (3 * d + d + d + d + 4 * d) / DC_CS;    // output rows of the K = d matrices in a slice
  p.w_layer = (rows_d * pw + (d / DC_CS) * pw4) * 2;
  int o = resident ? layers * p.w_layer : 0;     // not resident: weight slices are read from L2 where they are used
  auto take = [&](int bytes) { int r = o; o += (bytes + 15) & ~15; return r; };
  p.off_h = take(DC_ROWS * d * 4);
  p.off_a = take(DC_ROWS * (d + 8) * 2);
  p.off_qkv = take(DC_ROWS * (3 * d + 8) * 2);
  p.off_q2 = take(DC_ROWS * (d + 8) * 2);
  p.off_f = take(DC_ROWS * (4 * d + 8) * 2);
  p.off_red = take(DC_WARPS * DC_ROWS * 8 * 4);              // one 16 x 8 fp32 tile per warp
  p.off_kv = take((resident ? layers : 1) * DC_MAX_NK * 2 * d * 4);   // keys / values of the memory tokens: every block, or the current one
  p.off_x = take(DC_ROWS * 16 * 4 * 2);                      // latent and eps, D <= 256
  p.off_posb = take(DC_ROWS * d * 4);
  p.off_win = take(A * d * 4);
  p.off_par = take((layers * (7 * d + 11 * d / DC_CS) + 2 * d + A * d + 16) * 4);   // LayerNorm parameters, this CTA's bias slices, the whole bo2, head
  p.total = o;
  return p;
}

// Y[16, n_slice] = X[16, KD] * Wslice[n_slice, KD]^T.  Work units are (8-column tile, K part): with
// fewer tiles than warps the K range is split and the parts are summed through shared memory.
// `emit(row, col, v)` receives 8 adjacent columns (col a multiple of 8) of the finished slice.
__host__ __device__ constexpr int dc_ksplit(int KD, int n_tiles) {
  int ksplit = 1;
  while (n_tiles * ksplit * 2 <= DC_WARPS && (KD / 32) % (ksplit * 2) == 0) ksplit *= 2;     // parts of whole 32-k blocks
  return ksplit;
}
template <int KD, int NSLICE, typename Emit>
__device__ __forceinline__ void dc_linear(const __nv_bfloat16* X, int px, const __nv_bfloat16* W, int PW, float* red, Emit emit) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, tg = lane & 3;
  constexpr int n_tiles = NSLICE >> 3;      // PW: row pitch of W (KD + 8 in shared memory, KD in global memory)
  constexpr int ksplit = dc_ksplit(KD, n_tiles);
  constexpr int units = n_tiles * ksplit;
  if constexpr (ksplit == 1) {
    // No K split: a warp owns whole tiles (tiles warp, warp + 8, ...), so it finishes them on its own and the warps
    // run through the layer without meeting; one block barrier at the end.  All of a warp's tiles go through the k
    // loop together -- the activations are read once and the weight loads of every tile are in flight at the same
    // time -- then each is finished in turn: fragment to the warp's 16 x 8 patch of `red`, lanes 0..15 emit one row
    // each (same sums in the same order as the split path with one part).
    constexpr int TPW = (n_tiles + DC_WARPS - 1) / DC_WARPS;
    float* r = red + (size_t)warp * (DC_ROWS * 8);
    float c[TPW][4];
#pragma unroll
    for (int t = 0; t < TPW; ++t) { c[t][0] = c[t][1] = c[t][2] = c[t][3] = 0.f; }
    const __nv_bfloat16* x0 = X + (size_t)g * px;
    const __nv_bfloat16* x1 = X + (size_t)(g + 8) * px;
#pragma unroll 8
    for (int ks = 0; ks < KD / 16; ks += 2) {
      const int k = ks * 16 + 8 * tg;
      const uint4 xa = *reinterpret_cast<const uint4*>(x0 + k);
      const uint4 xb = *reinterpret_cast<const uint4*>(x1 + k);
      const uint32_t a1[4] = {xa.x, xb.x, xa.y, xb.y}, a2[4] = {xa.z, xb.z, xa.w, xb.w};
      uint4 wv[TPW];
#pragma unroll
      for (int t = 0; t < TPW; ++t) {
        const int nt = min(warp + t * DC_WARPS, n_tiles - 1);          // past the last tile: recomputed, not emitted
        wv[t] = *reinterpret_cast<const uint4*>(W + (size_t)(nt * 8 + g) * PW + k);
      }
#pragma unroll
      for (int t = 0; t < TPW; ++t) {
        mma_bf16_16816(c[t], a1, wv[t].x, wv[t].y);
        mma_bf16_16816(c[t], a2, wv[t].z, wv[t].w);
      }
    }
#pragma unroll
    for (int t = 0; t < TPW; ++t) {
      const int nt = warp + t * DC_WARPS;
      if (nt < n_tiles) {                                               // warp-uniform
        r[g * 8 + 2 * tg] = c[t][0]; r[g * 8 + 2 * tg + 1] = c[t][1];
        r[(g + 8) * 8 + 2 * tg] = c[t][2]; r[(g + 8) * 8 + 2 * tg + 1] = c[t][3];
        __syncwarp();
        if (lane < DC_ROWS) {
          const float4* rp = reinterpret_cast<const float4*>(r + lane * 8);
          const float4 lo = rp[0], hi = rp[1];
          float v[8] = {0.f + lo.x, 0.f + lo.y, 0.f + lo.z, 0.f + lo.w, 0.f + hi.x, 0.f + hi.y, 0.f + hi.z, 0.f + hi.w};
          emit(lane, nt * 8, v);
        }
        __syncwarp();
      }
    }
    __syncthreads();
  } else {
  for (int u0 = 0; u0 < units; u0 += DC_WARPS) {
    const int u = u0 + warp;
    if (u < units) {
      const int nt = u % n_tiles, kp = u / n_tiles;
      const int ks0 = kp * (KD / 16 / ksplit), ks1 = ks0 + KD / 16 / ksplit;
      float c[4] = {0.f, 0.f, 0.f, 0.f};
      const __nv_bfloat16* wrow = W + (size_t)(nt * 8 + g) * PW;
      const __nv_bfloat16* x0 = X + (size_t)g * px;
      const __nv_bfloat16* x1 = X + (size_t)(g + 8) * px;
      // Two k-steps (32 values of k) per iteration.  Lane (g, tg) reads 8 CONSECUTIVE k of its rows, 16 bytes at
      // a time, and feeds pairs (0,1 | 2,3) to the first mma and (4,5 | 6,7) to the second: a permutation of k
      // inside the block of 32 that A and B share, so the sum is unchanged while every load is one full
      // 16-byte access (four times fewer loads than the natural fragment layout; it matters most when the
      // weights come from the L2).
#pragma unroll 8
      for (int ks = ks0; ks < ks1; ks += 2) {
        const int k = ks * 16 + 8 * tg;
        const uint4 xa = *reinterpret_cast<const uint4*>(x0 + k);
        const uint4 xb = *reinterpret_cast<const uint4*>(x1 + k);
        const uint4 wv = *reinterpret_cast<const uint4*>(wrow + k);
        const uint32_t a1[4] = {xa.x, xb.x, xa.y, xb.y}, a2[4] = {xa.z, xb.z, xa.w, xb.w};
        mma_bf16_16816(c, a1, wv.x, wv.y);
        mma_bf16_16816(c, a2, wv.z, wv.w);
      }
      float* r = red + (size_t)warp * (DC_ROWS * 8);
      r[g * 8 + 2 * tg] = c[0]; r[g * 8 + 2 * tg + 1] = c[1];
      r[(g + 8) * 8 + 2 * tg] = c[2]; r[(g + 8) * 8 + 2 * tg + 1] = c[3];
    }
    __syncthreads();
    // finished tiles of this pass: tile nt = sum over its K parts (warps nt, nt + n_tiles, ...);
    // one thread finishes one row of one tile, so that it can store 8 adjacent columns at once
    const int tiles_here = min(n_tiles, DC_WARPS);   // units are laid out part-major: a pass holds whole tiles
    for (int i = threadIdx.x; i < tiles_here * DC_ROWS; i += DC_THREADS) {
      const int nt = i / DC_ROWS, row = i % DC_ROWS;
      const int tile = u0 + nt;              // with a K split there is a single pass (u0 = 0)
      if (tile >= n_tiles) continue;
      float v[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) v[j] = 0.f;
      for (int kp = 0; kp < ksplit; ++kp) {
        const float4* rp = reinterpret_cast<const float4*>(red + (size_t)(nt + kp * n_tiles) * (DC_ROWS * 8) + row * 8);
        const float4 lo = rp[0], hi = rp[1];
        v[0] += lo.x; v[1] += lo.y; v[2] += lo.z; v[3] += lo.w; v[4] += hi.x; v[5] += hi.y; v[6] += hi.z; v[7] += hi.w;
      }
      emit(row, tile * 8, v);
    }
    __syncthreads();
  }
  }
}


// LayerNorm of the 16 replicated rows: each half-warp normalises one row (warp w: rows 2w and 2w + 1), so
// the 16 rows go through in one pass; fp32 in, bf16 out.
__device__ __forceinline__ float half_warp_sum(float v) {
#pragma unroll
  for (int o = 8; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
template <int D_MODEL, bool AFFINE = true>
__device__ __forceinline__ void dc_layernorm(const float* h, const float* gam, const float* bet,
                                             __nv_bfloat16* out, int pitch) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int row = 2 * warp + (lane >> 4), l16 = lane & 15;
  constexpr int V = D_MODEL / 64;          // float4 per lane
  float4 v[V];
  float s = 0.f;
#pragma unroll
  for (int j = 0; j < V; ++j) {
    v[j] = *reinterpret_cast<const float4*>(h + row * D_MODEL + (j * 16 + l16) * 4);
    s += v[j].x + v[j].y + v[j].z + v[j].w;
  }
  const float mean = half_warp_sum(s) / D_MODEL;
  float q = 0.f;
#pragma unroll
  for (int j = 0; j < V; ++j) {
    v[j].x -= mean; v[j].y -= mean; v[j].z -= mean; v[j].w -= mean;
    q += v[j].x * v[j].x + v[j].y * v[j].y + v[j].z * v[j].z + v[j].w * v[j].w;
  }
  const float rstd = rsqrtf(half_warp_sum(q) / D_MODEL + 1e-5f);
#pragma unroll
  for (int j = 0; j < V; ++j) {
    const int c = (j * 16 + l16) * 4;
    if (AFFINE) {
      const float4 gg = *reinterpret_cast<const float4*>(gam + c), bb = *reinterpret_cast<const float4*>(bet + c);
      store4(out + row * pitch + c, v[j].x * rstd * gg.x + bb.x, v[j].y * rstd * gg.y + bb.y,
             v[j].z * rstd * gg.z + bb.z, v[j].w * rstd * gg.w + bb.w);
    } else {
      store4(out + row * pitch + c, v[j].x * rstd, v[j].y * rstd, v[j].z * rstd, v[j].w * rstd);
    }
  }
}

// Attention of the replicated sequence, recomputed by every CTA: four lanes own one (head, query row),
// each a quarter of the head width.  SELF: causal over the H tokens in qkv; otherwise over NK memory
// tokens whose keys/values are the fp32 rows kv[kx] = [K (d) | V (d)].
template <int D_MODEL, bool SELF>
__device__ __forceinline__ void dc_attention(const __nv_bfloat16* qsrc, int pq, const __nv_bfloat16* qkv, int pqkv,
                                             const float* kv, int NK, __nv_bfloat16* out, int po, int heads, int H) {
  const int dh = D_MODEL / heads, seg = dh >> 2;
  const int sub = threadIdx.x & 3;
  const float scale = rsqrtf((float)dh);
  for (int p = threadIdx.x >> 2; p < heads * DC_ROWS; p += DC_THREADS / 4) {
    const int head = p / DC_ROWS, row = p % DC_ROWS;
    const int c0 = head * dh + sub * seg;
    constexpr int NKEY = SELF ? DC_ROWS : DC_MAX_NK;
    float sc[NKEY];
    float m = -INFINITY;
#pragma unroll
    for (int j = 0; j < NKEY; ++j) {
      float a = 0.f;
      if (SELF) {
        for (int i = 0; i < seg; ++i)
          a += __bfloat162float(qsrc[row * pq + c0 + i]) * __bfloat162float(qkv[j * pqkv + D_MODEL + c0 + i]);
      } else if (j < NK) {
        for (int i = 0; i < seg; ++i) a += __bfloat162float(qsrc[row * pq + c0 + i]) * kv[j * 2 * D_MODEL + c0 + i];
      }
      a += __shfl_xor_sync(0xffffffffu, a, 1);
      a += __shfl_xor_sync(0xffffffffu, a, 2);
      const bool vis = SELF ? (j <= row && j < H) : (j < NK);
      sc[j] = vis ? a * scale : -INFINITY;
      m = fmaxf(m, sc[j]);
    }
    if (m == -INFINITY) m = 0.f;            // padding rows see nothing; keep them finite
    float l = 0.f;
#pragma unroll
    for (int j = 0; j < NKEY; ++j) { sc[j] = __expf(sc[j] - m); l += sc[j]; }
    const float inv = l > 0.f ? 1.0f / l : 0.f;
    for (int i = 0; i < seg; ++i) {
      float o = 0.f;
#pragma unroll
      for (int j = 0; j < NKEY; ++j) {
        if (SELF) o += sc[j] * __bfloat162float(qkv[j * pqkv + 2 * D_MODEL + c0 + i]);
        else if (j < NK) o += sc[j] * kv[j * 2 * D_MODEL + D_MODEL + c0 + i];
      }
      out[row * po + c0 + i] = __float2bfloat16_rn(o * inv);
    }
  }
}

// Causal self-attention of the replicated 16-token sequence on mma.sync: warp w takes heads w, w + 8, ...
// Same fragment algebra as self_attn_mma_kernel, operands read from the shared-memory qkv replica.
template <int D_MODEL, int DH>
__device__ __forceinline__ void dc_self_attn_mma(const __nv_bfloat16* qkv, int pqkv, __nv_bfloat16* out, int po, int heads,
                                                 int H) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, tg = lane & 3;
  constexpr int KS = DH / 16, NO = DH / 8;
  const float scale = rsqrtf((float)DH);
  for (int hd = warp; hd < heads; hd += DC_WARPS) {
    const __nv_bfloat16* qb = qkv + hd * DH;
    const __nv_bfloat16* kb = qkv + D_MODEL + hd * DH;
    const __nv_bfloat16* vb = qkv + 2 * D_MODEL + hd * DH;
    float s[2][4];
#pragma unroll
    for (int nt = 0; nt < 2; ++nt) {
      s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f;
#pragma unroll
      for (int ks = 0; ks < KS; ++ks) {
        const int k = ks * 16 + 2 * tg;
        uint32_t a[4];
        a[0] = *reinterpret_cast<const uint32_t*>(qb + g * pqkv + k);
        a[1] = *reinterpret_cast<const uint32_t*>(qb + (g + 8) * pqkv + k);
        a[2] = *reinterpret_cast<const uint32_t*>(qb + g * pqkv + k + 8);
        a[3] = *reinterpret_cast<const uint32_t*>(qb + (g + 8) * pqkv + k + 8);
        const uint32_t b0 = *reinterpret_cast<const uint32_t*>(kb + (nt * 8 + g) * pqkv + k);
        const uint32_t b1 = *reinterpret_cast<const uint32_t*>(kb + (nt * 8 + g) * pqkv + k + 8);
        mma_bf16_16816(s[nt], a, b0, b1);
      }
    }
    const int r0 = g, r1 = g + 8;
    float m0 = -INFINITY, m1 = -INFINITY;
#pragma unroll
    for (int nt = 0; nt < 2; ++nt) {
      const int col = nt * 8 + 2 * tg;
      s[nt][0] = (col <= r0 && col < H) ? s[nt][0] * scale : -INFINITY;
      s[nt][1] = (col + 1 <= r0 && col + 1 < H) ? s[nt][1] * scale : -INFINITY;
      s[nt][2] = (col <= r1 && col < H) ? s[nt][2] * scale : -INFINITY;
      s[nt][3] = (col + 1 <= r1 && col + 1 < H) ? s[nt][3] * scale : -INFINITY;
      m0 = fmaxf(m0, fmaxf(s[nt][0], s[nt][1]));
      m1 = fmaxf(m1, fmaxf(s[nt][2], s[nt][3]));
    }
    m0 = fmaxf(m0, __shfl_xor_sync(0xffffffffu, m0, 1)); m0 = fmaxf(m0, __shfl_xor_sync(0xffffffffu, m0, 2));
    m1 = fmaxf(m1, __shfl_xor_sync(0xffffffffu, m1, 1)); m1 = fmaxf(m1, __shfl_xor_sync(0xffffffffu, m1, 2));
    if (m0 == -INFINITY) m0 = 0.f;
    if (m1 == -INFINITY) m1 = 0.f;
    float l0 = 0.f, l1 = 0.f;
#pragma unroll
    for (int nt = 0; nt < 2; ++nt) {
      s[nt][0] = __expf(s[nt][0] - m0); s[nt][1] = __expf(s[nt][1] - m0);
      s[nt][2] = __expf(s[nt][2] - m1); s[nt][3] = __expf(s[nt][3] - m1);
      l0 += s[nt][0] + s[nt][1]; l1 += s[nt][2] + s[nt][3];
    }
    l0 += __shfl_xor_sync(0xffffffffu, l0, 1); l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 1); l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
    const float inv0 = l0 > 0.f ? 1.0f / l0 : 0.f, inv1 = l1 > 0.f ? 1.0f / l1 : 0.f;
    uint32_t pa[4];
    pa[0] = pack_bf16x2(s[0][0], s[0][1]); pa[1] = pack_bf16x2(s[0][2], s[0][3]);
    pa[2] = pack_bf16x2(s[1][0], s[1][1]); pa[3] = pack_bf16x2(s[1][2], s[1][3]);
    const unsigned short* vraw = reinterpret_cast<const unsigned short*>(vb);
#pragma unroll
    for (int no = 0; no < NO; ++no) {
      float o[4] = {0.f, 0.f, 0.f, 0.f};
      const int col = no * 8 + g, k0 = 2 * tg;
      const uint32_t b0 = (uint32_t)vraw[k0 * pqkv + col] | ((uint32_t)vraw[(k0 + 1) * pqkv + col] << 16);
      const uint32_t b1 = (uint32_t)vraw[(k0 + 8) * pqkv + col] | ((uint32_t)vraw[(k0 + 9) * pqkv + col] << 16);
      mma_bf16_16816(o, pa, b0, b1);
      const int oc = hd * DH + no * 8 + 2 * tg;
      *reinterpret_cast<uint32_t*>(out + r0 * po + oc) = pack_bf16x2(o[0] * inv0, o[1] * inv0);
      *reinterpret_cast<uint32_t*>(out + r1 * po + oc) = pack_bf16x2(o[2] * inv1, o[3] * inv1);
    }
  }
}

// Copy this CTA's block of `rows_per_cta` output rows of W [N, KD] into shared memory (row pitch KD + 8).
template <int KD>
__device__ __forceinline__ void dc_load_slice(__nv_bfloat16* dst, const __nv_bfloat16* __restrict__ W, int rows_per_cta,
                                              int rank) {
  constexpr int VPR = KD / 8;                      // 16-byte vectors per row
  const uint4* src = reinterpret_cast<const uint4*>(W + (size_t)rank * rows_per_cta * KD);
  for (int i = threadIdx.x; i < rows_per_cta * VPR; i += DC_THREADS) {
    const int r = i / VPR, v = i % VPR;
    *reinterpret_cast<uint4*>(dst + (size_t)r * (KD + 8) + v * 8) = __ldg(src + (size_t)r * VPR + v);
  }
}

template <int D_MODEL>
__global__ void __cluster_dims__(DC_CS, 1, 1) __launch_bounds__(DC_THREADS, 1)
drafter_cluster_kernel(const __grid_constant__ DcParams P) {
  extern __shared__ __align__(16) uint8_t dc_smem[];
  pdl_trigger();
  cg::cluster_group cluster = cg::this_cluster();
  const int rank = (int)cluster.block_rank();
  const int cid = blockIdx.x / DC_CS, ncl = gridDim.x / DC_CS;
  // stage hand-over: two mbarriers that count the bytes of the slices arriving in this CTA (see the file header)
  __shared__ __align__(8) uint64_t dc_bar[2];
  const bool use_async = P.async_bcast != 0;
  const uint32_t bar_addr[2] = {ptx::smem_u32(&dc_bar[0]), ptx::smem_u32(&dc_bar[1])};
  if (threadIdx.x == 0) {
    ptx::mbar_init(bar_addr[0], 1);
    ptx::mbar_init(bar_addr[1], 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  uint32_t stage_no = 0, stage_phase = 0;      // stages so far; bit b = parity this CTA waits for next on barrier b
  bool wait_failed = false;
  // thread 0 announces the bytes this CTA will receive in the stage that begins
  auto stage_begin = [&](uint32_t bytes) {
    if (use_async && threadIdx.x == 0)
      asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar_addr[stage_no & 1u]), "r"(bytes) : "memory");
  };
  // 16 bytes to the same shared-memory address in every CTA of the cluster
  auto bcast16 = [&](const void* local_ptr, const uint4& v) {
    const uint32_t la = ptx::smem_u32(local_ptr);
    if (use_async) {
      const uint32_t lb = bar_addr[stage_no & 1u];
#pragma unroll
      for (uint32_t r = 0; r < DC_CS; ++r) dc_st_async16(dc_mapa(la, r), v, dc_mapa(lb, r));
    } else {
#pragma unroll 1
      for (uint32_t r = 0; r < DC_CS; ++r) dc_st_cluster16(dc_mapa(la, r), v);
    }
  };
  // every slice of the stage has arrived in this CTA (bounded wait), or, without st.async, the cluster barrier
  auto stage_end = [&]() {
    if (use_async) {
      const uint32_t b = stage_no & 1u, par = (stage_phase >> b) & 1u;
      uint32_t done = wait_failed ? 1u : 0u;       // after one wait has given up the rest of the launch does not wait again
      const long long t0 = clock64();
      while (!done) {
        asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
                     : "=r"(done) : "r"(bar_addr[b]), "r"(par) : "memory");
        if (!done && clock64() - t0 > GEMM_WAIT_CYCLES) {      // about a second: report, and run to the end without waiting
          wait_failed = true;
          if (threadIdx.x == 0) atomicExch(P.status, 5);
          break;
        }
      }
      stage_phase ^= 1u << b;
      ++stage_no;
    } else {
      cluster.sync();
    }
  };
  constexpr int d = D_MODEL;
  constexpr int PA = d + 8, PQKV = 3 * d + 8, PF = 4 * d + 8;
  const bool resident = P.resident != 0;
  const DcSmem pl = dc_smem_plan(d, P.layers, P.A, resident);
  float* h = reinterpret_cast<float*>(dc_smem + pl.off_h);
  __nv_bfloat16* a = reinterpret_cast<__nv_bfloat16*>(dc_smem + pl.off_a);
  __nv_bfloat16* qkv = reinterpret_cast<__nv_bfloat16*>(dc_smem + pl.off_qkv);
  __nv_bfloat16* q2 = reinterpret_cast<__nv_bfloat16*>(dc_smem + pl.off_q2);
  __nv_bfloat16* f = reinterpret_cast<__nv_bfloat16*>(dc_smem + pl.off_f);
  float* red = reinterpret_cast<float*>(dc_smem + pl.off_red);
  float* skv = reinterpret_cast<float*>(dc_smem + pl.off_kv);
  float* sx = reinterpret_cast<float*>(dc_smem + pl.off_x);
  float* seps = sx + DC_ROWS * 16;
  float* posb = reinterpret_cast<float*>(dc_smem + pl.off_posb);
  float* win = reinterpret_cast<float*>(dc_smem + pl.off_win);
  float* par = reinterpret_cast<float*>(dc_smem + pl.off_par);
  const int H = P.H, A = P.A, D = H * A, L = P.layers, NK = 1 + P.To;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  // ---- once per launch: this CTA's weight slices, embedding tables, zeroed activations
  constexpr int NS_D = d / DC_CS, NS_3D = 3 * d / DC_CS, NS_4D = 4 * d / DC_CS;   // slice widths
  auto w_ptr = [&](int l, int which) -> const __nv_bfloat16* {     // 0 qkv, 1 o, 2 q2, 3 o2, 4 w1, 5 w2
    if (!resident) {      // this CTA's block of output rows, in place in global memory (served by the L2)
      const DcLayer& G = P.L[l];
      const __nv_bfloat16* base[6] = {G.Wqkv, G.Wo, G.Wq2, G.Wo2, G.W1, G.W2};
      const int rows[6] = {NS_3D, NS_D, NS_D, NS_D, NS_4D, NS_D};
      return base[which] + (size_t)rank * rows[which] * (which == 5 ? 4 * d : d);
    }
    const int rows_before[6] = {0, NS_3D, NS_3D + NS_D, NS_3D + 2 * NS_D, NS_3D + 3 * NS_D, NS_3D + 3 * NS_D + NS_4D};
    return reinterpret_cast<const __nv_bfloat16*>(dc_smem + (size_t)l * pl.w_layer) + (size_t)rows_before[which] * PA;
  };
  const int PWD = resident ? PA : d, PW4 = resident ? PF : 4 * d;      // weight row pitches for K = d and K = 4d
  for (int l = 0; l < L && resident; ++l) {
    dc_load_slice<d>(const_cast<__nv_bfloat16*>(w_ptr(l, 0)), P.L[l].Wqkv, NS_3D, rank);
    dc_load_slice<d>(const_cast<__nv_bfloat16*>(w_ptr(l, 1)), P.L[l].Wo, NS_D, rank);
    dc_load_slice<d>(const_cast<__nv_bfloat16*>(w_ptr(l, 2)), P.L[l].Wq2, NS_D, rank);
    dc_load_slice<d>(const_cast<__nv_bfloat16*>(w_ptr(l, 3)), P.L[l].Wo2, NS_D, rank);
    dc_load_slice<d>(const_cast<__nv_bfloat16*>(w_ptr(l, 4)), P.L[l].W1, NS_4D, rank);
    dc_load_slice<4 * d>(const_cast<__nv_bfloat16*>(w_ptr(l, 5)), P.L[l].W2, NS_D, rank);
  }
  for (int i = threadIdx.x; i < DC_ROWS * d; i += DC_THREADS) {
    const int row = i / d, col = i % d;
    posb[i] = row < H ? P.b_in[col] + P.pos[row * d + col] : 0.f;
    h[i] = 0.f;
  }
  for (int i = threadIdx.x; i < A * d; i += DC_THREADS) win[i] = P.W_in[i];
  // LayerNorm parameters and this CTA's slices of the biases of every block, then the head: read from shared
  // memory on the critical path
  constexpr int PL = 7 * d + 11 * d / DC_CS;       // floats per block: 6 LayerNorm vectors, bias slices, the whole bo2
  for (int l = 0; l < L; ++l) {
    const DcLayer& G = P.L[l];
    const float* ln[6] = {G.ln1_g, G.ln1_b, G.ln2_g, G.ln2_b, G.ln3_g, G.ln3_b};
    for (int j = 0; j < 6; ++j)
      for (int i = threadIdx.x; i < d; i += DC_THREADS) par[(size_t)l * PL + j * d + i] = ln[j][i];
    const float* bs[6] = {G.bqkv, G.bo, G.bq2, G.bo2, G.b1, G.b2};
    const int ns[6] = {3 * d / DC_CS, d / DC_CS, d / DC_CS, d / DC_CS, 4 * d / DC_CS, d / DC_CS};
    int off = 6 * d;
    for (int j = 0; j < 6; ++j) {
      for (int i = threadIdx.x; i < ns[j]; i += DC_THREADS) par[(size_t)l * PL + off + i] = bs[j][rank * ns[j] + i];
      off += ns[j];
    }
    for (int i = threadIdx.x; i < d; i += DC_THREADS) par[(size_t)l * PL + off + i] = G.bo2[i];
  }
  float* lnf_g = par + (size_t)L * PL;
  float* lnf_b = lnf_g + d;
  float* woutT = lnf_b + d;
  float* bout = woutT + A * d;
  for (int i = threadIdx.x; i < d; i += DC_THREADS) { lnf_g[i] = P.lnf_g[i]; lnf_b[i] = P.lnf_b[i]; }
  for (int i = threadIdx.x; i < A * d; i += DC_THREADS) woutT[i] = P.W_outT[i];
  for (int i = threadIdx.x; i < A; i += DC_THREADS) bout[i] = P.b_out[i];
  for (int i = threadIdx.x; i < DC_ROWS * PA; i += DC_THREADS) { a[i] = __float2bfloat16_rn(0.f); q2[i] = a[i]; }
  for (int i = threadIdx.x; i < DC_ROWS * PQKV; i += DC_THREADS) qkv[i] = __float2bfloat16_rn(0.f);
  for (int i = threadIdx.x; i < DC_ROWS * PF; i += DC_THREADS) f[i] = __float2bfloat16_rn(0.f);
  // The replicas of the other CTAs are addressed through distributed shared memory (map_shared_rank in a rolled
  // loop at each broadcast: the kernel is a long straight line of code executed once per stage, so code size
  // -- instruction-cache misses -- matters more than the few address computations).
  cluster.sync();
  pdl_wait();      // weights and tables above are constant; t, the latents and the obs K/V come from earlier kernels

  const uint64_t seed = *P.seed;
  const size_t ldkv = (size_t)L * 2 * d;
  // One forward of the network on the latent in sx at timestep tau for request env; leaves eps in seps.
  auto forward = [&](int tau, int env) {
    // keys / values of the time token of tau, every block
    for (int i = threadIdx.x; i < (resident && !P.fold ? L : 0) * 2 * d; i += DC_THREADS) {
      const int l = i / (2 * d), c = i % (2 * d);
      skv[(size_t)l * DC_MAX_NK * 2 * d + c] = __ldg(P.kv_time + (size_t)tau * ldkv + (size_t)l * 2 * d + c);
    }
    // token embedding into the residual stream
    for (int i = threadIdx.x; i < DC_ROWS * d; i += DC_THREADS) {
      const int row = i / d, col = i % d;
      float v = posb[i];
      if (row < H)
        for (int c = 0; c < A; ++c) v += sx[row * A + c] * win[c * d + col];
      h[i] = v;
    }
    __syncthreads();
    for (int l = 0; l < L; ++l) {
      const float* pb = par + (size_t)l * PL;
      const float* bb = pb + 6 * d;                      // bias slices: columns of this CTA only
      struct { const float *ln1_g, *ln1_b, *ln2_g, *ln2_b, *ln3_g, *ln3_b, *bqkv, *bo, *bq2, *bo2, *b1, *b2; } W =
          {pb, pb + d, pb + 2 * d, pb + 3 * d, pb + 4 * d, pb + 5 * d, bb, bb + NS_3D, bb + NS_3D + NS_D,
           bb + NS_3D + 2 * NS_D, bb + NS_3D + 3 * NS_D, bb + NS_3D + 3 * NS_D + NS_4D};
      // ---- causal self-attention
      dc_layernorm<d>(h, W.ln1_g, W.ln1_b, a, PA);
      __syncthreads();
      stage_begin(DC_ROWS * 3 * d * 2);
      dc_linear<d, NS_3D>(a, PA, w_ptr(l, 0), PWD, red, [&](int row, int col, float* v) {
        const int cg_ = rank * NS_3D + col;
        const float4 b0 = *reinterpret_cast<const float4*>(W.bqkv + col), b1 = *(reinterpret_cast<const float4*>(W.bqkv + col) + 1);
        v[0] += b0.x; v[1] += b0.y; v[2] += b0.z; v[3] += b0.w; v[4] += b1.x; v[5] += b1.y; v[6] += b1.z; v[7] += b1.w;
        const uint4 pk = make_uint4(pack_bf16x2(v[0], v[1]), pack_bf16x2(v[2], v[3]), pack_bf16x2(v[4], v[5]), pack_bf16x2(v[6], v[7]));
        bcast16(qkv + row * PQKV + cg_, pk);
      });
      stage_end();
      switch (d / P.heads) {
        case 32: dc_self_attn_mma<d, 32>(qkv, PQKV, a, PA, P.heads, H); break;
        case 64: dc_self_attn_mma<d, 64>(qkv, PQKV, a, PA, P.heads, H); break;
        case 128: dc_self_attn_mma<d, 128>(qkv, PQKV, a, PA, P.heads, H); break;
        default: dc_attention<d, true>(qkv, PQKV, qkv, PQKV, nullptr, 0, a, PA, P.heads, H); break;
      }
      __syncthreads();
      if (P.fold) {
        // the memory tokens' folded tables of this block start their way into shared memory now (the qkv buffer
        // is free until the next block, the q2 buffer is not used at all): kq rows with their constant in the
        // row padding -> q2 buffer; u rows as they are stored (head pairs in one word) -> qkv buffer
        const int heads = P.heads, hp = heads >> 1, NKH = NK * heads;
        const size_t tok_stride = (size_t)L * heads * d, lay = (size_t)l * heads * d;
        for (int i = threadIdx.x; i < NKH * (d / 8); i += DC_THREADS) {
          const int n = i / (d / 8), ch = i % (d / 8);
          const int j = n / heads, hh = n - j * heads;
          const __nv_bfloat16* src = (j == 0 ? P.kq_time + (size_t)tau * tok_stride : P.kq_obs + ((size_t)env * P.To + (j - 1)) * tok_stride) +
                                     lay + (size_t)hh * d + ch * 8;
          dc_cp_async<16>(q2 + n * PA + ch * 8, src);
        }
        for (int n = threadIdx.x; n < NKH; n += DC_THREADS) {
          const int j = n / heads, hh = n - j * heads;
          const float* src = (j == 0 ? P.c_time + (size_t)tau * L * heads : P.c_obs + ((size_t)env * P.To + (j - 1)) * L * heads) +
                             (size_t)l * heads + hh;
          dc_cp_async<4>(q2 + n * PA + d, src);
        }
        uint32_t* sU = reinterpret_cast<uint32_t*>(qkv);                    // [NKH / 2][d + 8] words: word (pair row, o) = u of heads 2q, 2q+1 at output column o
        for (int i = threadIdx.x; i < (NKH / 2) * (d / 4); i += DC_THREADS) {
          const int pr = i / (d / 4), ch = i - pr * (d / 4);
          const int j = pr / hp, q = pr - j * hp;
          const __nv_bfloat16* src = (j == 0 ? P.ut_time + (size_t)tau * tok_stride : P.ut_obs + ((size_t)env * P.To + (j - 1)) * tok_stride) +
                                     lay + (size_t)q * d * 2 + ch * 8;
          dc_cp_async<16>(sU + pr * (d + 8) + ch * 4, src);
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
      }
      stage_begin(DC_ROWS * d * 4);
      dc_linear<d, NS_D>(a, PA, w_ptr(l, 1), PWD, red, [&](int row, int col, float* v) {
        const int cg_ = rank * NS_D + col;
        const float4* hp = reinterpret_cast<const float4*>(h + row * d + cg_);
        const float4 h0 = hp[0], h1 = hp[1];
        const float4 b0 = *reinterpret_cast<const float4*>(W.bo + col), b1 = *(reinterpret_cast<const float4*>(W.bo + col) + 1);
        const float4 o0 = make_float4(h0.x + v[0] + b0.x, h0.y + v[1] + b0.y, h0.z + v[2] + b0.z, h0.w + v[3] + b0.w);
        const float4 o1 = make_float4(h1.x + v[4] + b1.x, h1.y + v[5] + b1.y, h1.z + v[6] + b1.z, h1.w + v[7] + b1.w);
        bcast16(h + row * d + cg_, make_uint4(__float_as_uint(o0.x), __float_as_uint(o0.y), __float_as_uint(o0.z), __float_as_uint(o0.w)));
        bcast16(h + row * d + cg_ + 4, make_uint4(__float_as_uint(o1.x), __float_as_uint(o1.y), __float_as_uint(o1.z), __float_as_uint(o1.w)));
      });
      if (!resident && !P.fold) {   // keys / values of the memory tokens for this block only: time token of tau, then the obs tokens
        for (int i = threadIdx.x; i < NK * 2 * d; i += DC_THREADS) {
          const int kx = i / (2 * d), c = i % (2 * d);
          const float* src = kx == 0 ? P.kv_time + (size_t)tau * ldkv : P.kv_obs + ((size_t)env * P.To + (kx - 1)) * ldkv;
          skv[i] = __ldg(src + (size_t)l * 2 * d + c);
        }
      }
      stage_end();
      if (use_async && !resident && !P.fold) __syncthreads();      // the keys / values above were written by other threads
      // ---- cross-attention to [time token | obs tokens]
      if (P.fold) {
        // Folded form: scores = xhat . kq + c, out = P . u + bo2, both so small that every CTA computes them whole
        // on its own replica: no slices to exchange, no cluster barrier, two linear stages fewer per block.
        const int heads = P.heads, NKH = NK * heads;
        float* sS = reinterpret_cast<float*>(qkv + (size_t)d * DC_PU);       // [16][16] scores
        __nv_bfloat16* sP = reinterpret_cast<__nv_bfloat16*>(sS + DC_ROWS * 16);   // [16][DC_PU] softmax weights
        dc_layernorm<d, false>(h, nullptr, nullptr, a, PA);
        for (int i = threadIdx.x; i < DC_ROWS * DC_PU / 2; i += DC_THREADS) reinterpret_cast<uint32_t*>(sP)[i] = 0u;
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        __syncthreads();
        dc_linear<d, 16>(a, PA, q2, PA, red, [&](int row, int col, float* v) {
#pragma unroll
          for (int j = 0; j < 8; ++j) sS[row * 16 + col + j] = v[j];
        });
        __syncthreads();
        for (int p = threadIdx.x; p < DC_ROWS * heads; p += DC_THREADS) {
          const int row = p / heads, hh = p - row * heads;
          float sc[DC_MAX_NK];
          float m = -INFINITY;
#pragma unroll
          for (int j = 0; j < DC_MAX_NK; ++j)
            if (j < NK) {
              const int n = j * heads + hh;
              sc[j] = sS[row * 16 + n] + *reinterpret_cast<const float*>(q2 + n * PA + d);
              m = fmaxf(m, sc[j]);
            }
          float lsum = 0.f;
#pragma unroll
          for (int j = 0; j < DC_MAX_NK; ++j)
            if (j < NK) { sc[j] = __expf(sc[j] - m); lsum += sc[j]; }
          const float inv = 1.0f / lsum;
#pragma unroll
          for (int j = 0; j < DC_MAX_NK; ++j)
            if (j < NK) sP[row * DC_PU + j * heads + hh] = __float2bfloat16_rn(sc[j] * inv);
        }
        __syncthreads();
        const float* bo2_full = pb + 6 * d + 11 * d / DC_CS;
        {
          // out = P . u: warp w the output columns [w d/8, (w+1) d/8), every row; a word of the u rows is one B
          // fragment register (k = heads 2q, 2q+1 of a memory token), so nothing is transposed.
          const int g = lane >> 2, tg = lane & 3;
          const uint32_t* sU = reinterpret_cast<const uint32_t*>(qkv);
          uint32_t pa[2][4];
#pragma unroll
          for (int k2 = 0; k2 < 2; ++k2) ldmatrix_x4(pa[k2], sP + (lane & 15) * DC_PU + k2 * 16 + 8 * (lane >> 4));
          const uint32_t* pu[2][2];
          uint32_t ulive[2][2];
#pragma unroll
          for (int k2 = 0; k2 < 2; ++k2)
#pragma unroll
            for (int rg = 0; rg < 2; ++rg) {
              const int pr = 8 * k2 + 4 * rg + tg;
              ulive[k2][rg] = 2 * pr < NKH ? 0xffffffffu : 0u;
              pu[k2][rg] = sU + (size_t)min(pr, NKH / 2 - 1) * (d + 8) + g;
            }
#pragma unroll
          for (int nt = 0; nt < d / 64; ++nt) {
            const int col = warp * (d / 8) + nt * 8;
            float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int k2 = 0; k2 < 2; ++k2)
              if (16 * k2 < NKH) mma_bf16_16816(acc, pa[k2], pu[k2][0][col] & ulive[k2][0], pu[k2][1][col] & ulive[k2][1]);
            // every CTA updates its own replica of the stream: straight from the fragment, two columns per lane and row
            const float2 b2 = *reinterpret_cast<const float2*>(bo2_full + col + 2 * tg);
            float2* h0 = reinterpret_cast<float2*>(h + g * d + col + 2 * tg);
            float2* h1 = reinterpret_cast<float2*>(h + (g + 8) * d + col + 2 * tg);
            float2 a0 = *h0, a1 = *h1;
            a0.x += acc[0] + b2.x; a0.y += acc[1] + b2.y; a1.x += acc[2] + b2.x; a1.y += acc[3] + b2.y;
            *h0 = a0; *h1 = a1;
          }
        }
        __syncthreads();
      } else {
      dc_layernorm<d>(h, W.ln2_g, W.ln2_b, a, PA);
      __syncthreads();
      stage_begin(DC_ROWS * d * 2);
      dc_linear<d, NS_D>(a, PA, w_ptr(l, 2), PWD, red, [&](int row, int col, float* v) {
        const int cg_ = rank * NS_D + col;
        const float4 b0 = *reinterpret_cast<const float4*>(W.bq2 + col), b1 = *(reinterpret_cast<const float4*>(W.bq2 + col) + 1);
        v[0] += b0.x; v[1] += b0.y; v[2] += b0.z; v[3] += b0.w; v[4] += b1.x; v[5] += b1.y; v[6] += b1.z; v[7] += b1.w;
        const uint4 pk = make_uint4(pack_bf16x2(v[0], v[1]), pack_bf16x2(v[2], v[3]), pack_bf16x2(v[4], v[5]), pack_bf16x2(v[6], v[7]));
        bcast16(q2 + row * PA + cg_, pk);
      });
      stage_end();
      dc_attention<d, false>(q2, PA, nullptr, 0, skv + (size_t)(resident ? l : 0) * DC_MAX_NK * 2 * d, NK, a, PA, P.heads, H);
      __syncthreads();
      stage_begin(DC_ROWS * d * 4);
      dc_linear<d, NS_D>(a, PA, w_ptr(l, 3), PWD, red, [&](int row, int col, float* v) {
        const int cg_ = rank * NS_D + col;
        const float4* hp = reinterpret_cast<const float4*>(h + row * d + cg_);
        const float4 h0 = hp[0], h1 = hp[1];
        const float4 b0 = *reinterpret_cast<const float4*>(W.bo2 + col), b1 = *(reinterpret_cast<const float4*>(W.bo2 + col) + 1);
        const float4 o0 = make_float4(h0.x + v[0] + b0.x, h0.y + v[1] + b0.y, h0.z + v[2] + b0.z, h0.w + v[3] + b0.w);
        const float4 o1 = make_float4(h1.x + v[4] + b1.x, h1.y + v[5] + b1.y, h1.z + v[6] + b1.z, h1.w + v[7] + b1.w);
        bcast16(h + row * d + cg_, make_uint4(__float_as_uint(o0.x), __float_as_uint(o0.y), __float_as_uint(o0.z), __float_as_uint(o0.w)));
        bcast16(h + row * d + cg_ + 4, make_uint4(__float_as_uint(o1.x), __float_as_uint(o1.y), __float_as_uint(o1.z), __float_as_uint(o1.w)));
      });
      stage_end();
      }
      // ---- MLP
      dc_layernorm<d>(h, W.ln3_g, W.ln3_b, a, PA);
      __syncthreads();
      stage_begin(DC_ROWS * 4 * d * 2);
      dc_linear<d, NS_4D>(a, PA, w_ptr(l, 4), PWD, red, [&](int row, int col, float* v) {
        const int cg_ = rank * NS_4D + col;
        const float4 b0 = *reinterpret_cast<const float4*>(W.b1 + col), b1 = *(reinterpret_cast<const float4*>(W.b1 + col) + 1);
        v[0] += b0.x; v[1] += b0.y; v[2] += b0.z; v[3] += b0.w; v[4] += b1.x; v[5] += b1.y; v[6] += b1.z; v[7] += b1.w;
#pragma unroll
        for (int j = 0; j < 8; ++j)
          v[j] = ptx::gelu_fast(v[j]);
        const uint4 pk = make_uint4(pack_bf16x2(v[0], v[1]), pack_bf16x2(v[2], v[3]), pack_bf16x2(v[4], v[5]), pack_bf16x2(v[6], v[7]));
        bcast16(f + row * PF + cg_, pk);
      });
      stage_end();
      stage_begin(DC_ROWS * d * 4);
      dc_linear<4 * d, NS_D>(f, PF, w_ptr(l, 5), PW4, red, [&](int row, int col, float* v) {
        const int cg_ = rank * NS_D + col;
        const float4* hp = reinterpret_cast<const float4*>(h + row * d + cg_);
        const float4 h0 = hp[0], h1 = hp[1];
        const float4 b0 = *reinterpret_cast<const float4*>(W.b2 + col), b1 = *(reinterpret_cast<const float4*>(W.b2 + col) + 1);
        const float4 o0 = make_float4(h0.x + v[0] + b0.x, h0.y + v[1] + b0.y, h0.z + v[2] + b0.z, h0.w + v[3] + b0.w);
        const float4 o1 = make_float4(h1.x + v[4] + b1.x, h1.y + v[5] + b1.y, h1.z + v[6] + b1.z, h1.w + v[7] + b1.w);
        bcast16(h + row * d + cg_, make_uint4(__float_as_uint(o0.x), __float_as_uint(o0.y), __float_as_uint(o0.z), __float_as_uint(o0.w)));
        bcast16(h + row * d + cg_ + 4, make_uint4(__float_as_uint(o1.x), __float_as_uint(o1.y), __float_as_uint(o1.z), __float_as_uint(o1.w)));
      });
      stage_end();
    }
    // ---- head: eps = LN_f(h) W_out + b_out   (every CTA, rows w and w + 8 per warp)
    {
      constexpr int V = d / 128;
#pragma unroll
      for (int rr = 0; rr < 2; ++rr) {
        const int row = warp + rr * 8;
        float4 v[V];
        float s = 0.f;
#pragma unroll
        for (int j = 0; j < V; ++j) {
          v[j] = *reinterpret_cast<const float4*>(h + row * d + j * 128 + lane * 4);
          s += v[j].x + v[j].y + v[j].z + v[j].w;
        }
        const float mean = warp_sum(s) / d;
        float q = 0.f;
#pragma unroll
        for (int j = 0; j < V; ++j) {
          v[j].x -= mean; v[j].y -= mean; v[j].z -= mean; v[j].w -= mean;
          q += v[j].x * v[j].x + v[j].y * v[j].y + v[j].z * v[j].z + v[j].w * v[j].w;
        }
        const float rstd = rsqrtf(warp_sum(q) / d + 1e-5f);
#pragma unroll
        for (int j = 0; j < V; ++j) {
          const int c = j * 128 + lane * 4;
          const float4 gg = *reinterpret_cast<const float4*>(lnf_g + c), bb = *reinterpret_cast<const float4*>(lnf_b + c);
          v[j].x = v[j].x * rstd * gg.x + bb.x; v[j].y = v[j].y * rstd * gg.y + bb.y;
          v[j].z = v[j].z * rstd * gg.z + bb.z; v[j].w = v[j].w * rstd * gg.w + bb.w;
        }
        for (int c = 0; c < A; ++c) {
          float acc = 0.f;
#pragma unroll
          for (int j = 0; j < V; ++j) {
            const float4 w = *reinterpret_cast<const float4*>(woutT + (size_t)c * d + j * 128 + lane * 4);
            acc += v[j].x * w.x + v[j].y * w.y + v[j].z * w.z + v[j].w * w.w;
          }
          acc = warp_sum(acc);
          if (lane == 0 && row < H) seps[row * A + c] = acc + bout[c];
        }
      }
    }
    __syncthreads();
  };

  if (P.mode == 1) {      // verification: one forward per (slot, candidate), the whole batch in one wave of clusters
    for (int w = cid; w < P.B * P.C; w += ncl) {
      const int slot = w / P.C, cand = w % P.C;
      const int tb = P.t[slot];
      if (tb < 0 || cand > tb) continue;          // finished slot, or a candidate beyond t = 0 (same for every CTA)
      const int env = item_of(P.item, slot);
      const float* xin = P.xt + slot * P.xs_b + (long long)cand * D;
      for (int i = threadIdx.x; i < D; i += DC_THREADS) sx[i] = xin[i];
      for (int i = threadIdx.x; i < (resident ? L : 0) * P.To * 2 * d; i += DC_THREADS) {
        const int l = i / (P.To * 2 * d), rem = i % (P.To * 2 * d);
        const int kx = 1 + rem / (2 * d), c = rem % (2 * d);
        skv[((size_t)l * DC_MAX_NK + kx) * 2 * d + c] = __ldg(P.kv_obs + ((size_t)env * P.To + (kx - 1)) * ldkv + (size_t)l * 2 * d + c);
      }
      __syncthreads();
      forward(tb - cand, env);
      if (rank == 0)
        for (int i = threadIdx.x; i < D; i += DC_THREADS) P.eps[slot * P.es_b + (long long)cand * D + i] = seps[i];
      __syncthreads();
    }
    cluster.sync();
    return;
  }
  for (int slot = cid; slot < P.B; slot += ncl) {
    const int tb = P.t[slot];
    const int env = item_of(P.item, slot);     // request served by this slot: its noise streams, obs K/V, parameters
    float* xt_b = P.xt + slot * P.xs_b;
    float* mh_b = P.muhat + slot * P.ms_b;
    for (int i = threadIdx.x; i < D; i += DC_THREADS) sx[i] = xt_b[i];
    // keys / values of this environment's observation tokens, every block (slot 0 is the time token)
    for (int i = threadIdx.x; i < (resident ? L : 0) * P.To * 2 * d; i += DC_THREADS) {
      const int l = i / (P.To * 2 * d), rem = i % (P.To * 2 * d);
      const int kx = 1 + rem / (2 * d), c = rem % (2 * d);
      skv[((size_t)l * DC_MAX_NK + kx) * 2 * d + c] = __ldg(P.kv_obs + ((size_t)env * P.To + (kx - 1)) * ldkv + (size_t)l * 2 * d + c);
    }
    __syncthreads();
    for (int k = 1; k <= P.K; ++k) {
      const int tau = tb - k + 1;
      if (!(tb >= 0 && tau >= 1 && k <= env_draft_cap(P.envp, env, tb, P.K, P.T))) {          // beyond K_eff: carry the latent along (same for every CTA)
        if (rank == 0)
          for (int i = threadIdx.x; i < D; i += DC_THREADS) {
            mh_b[(size_t)(k - 1) * D + i] = sx[i];
            xt_b[(size_t)k * D + i] = sx[i];
          }
        continue;
      }
      forward(tau, env);
      // ---- scheduler step: mu^_k, x~_k = mu^_k + sigma_tau xi_tau
      {
        const int nq = (D + 3) >> 2;
        for (int q = threadIdx.x; q < nq; q += DC_THREADS) {
          float z[4];
          normal4(seed, (uint32_t)env, STREAM_XI, (uint32_t)tau, (uint32_t)q, z);
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const int i = 4 * q + j;
            if (i < D) {
              const float m = posterior_mean(P.S, sx[i], seps[i], tau);
              const float xn = ddpm_sample(m, P.S.sigma[tau], z[j]);
              sx[i] = xn;
              if (rank == 0) { mh_b[(size_t)(k - 1) * D + i] = m; xt_b[(size_t)k * D + i] = xn; }
            }
          }
        }
      }
      __syncthreads();
    }
    __syncthreads();
  }
  cluster.sync();      // no CTA leaves while another may still write into its shared memory
}
}  // namespace tsdp
