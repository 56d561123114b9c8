// bf16 GEMM for sm_100a:  C[M,N] = A[M,K] * W[N,K]^T (+ bias, activation, residual), fp32 accumulate.
//
// This is the dense contraction of the verification forward (Sec. 3.2, "evaluating the frozen
// target model on all elements of C in a single batched forward pass"): every linear layer of the
// base transformer applied to all (K+1)*B candidate latents at once.
//
// Structure (one persistent CTA per SM, 128 x BN output tiles, BK = 64):
//   warp 0      TMA producer: cp.async.bulk.tensor 2-D tiles of A and W (both K-major, 128-byte
//               swizzle) into a ring of shared-memory stages, completion on mbarriers.
//   warp 1      MMA issuer: one elected thread issues tcgen05.mma (128 x BN x 16, kind::f16, bf16
//               inputs) into one of two TMEM accumulator buffers; tcgen05.commit releases smem
//               stages and publishes finished accumulators.
//   warps 2..9  epilogue: tcgen05.ld the accumulator (each warp owns one 32-lane TMEM quadrant and
//               half of the columns), fuse bias / GELU / residual, store.  The second accumulator
//               buffer lets the next tile's MMAs overlap this tile's epilogue.
// Every mbarrier wait is bounded: on expiry the kernel records TSDP_ERR_TIMEOUT in `status`, drains,
// frees its TMEM and returns.  No cluster launch, no multicast.
#pragma once
#include <cuda.h>
#include "common.cuh"

namespace tsdp {

enum { EPI_STORE = 0, EPI_GELU = 1, EPI_RESID = 2, EPI_F32 = 3 };

constexpr int GEMM_BM = 128;
constexpr int GEMM_BK = 64;
constexpr int GEMM_THREADS = 320;
constexpr int GEMM_EPI_WARPS = 8;
constexpr long long GEMM_WAIT_CYCLES = 2000000000ll;   // about one second of SM clock

__host__ __device__ constexpr int gemm_stages(int BN) { return BN >= 256 ? 4 : (BN >= 128 ? 6 : 8); }
__host__ __device__ constexpr int gemm_stage_bytes(int BN) { return GEMM_BM * GEMM_BK * 2 + BN * GEMM_BK * 2; }
__host__ __device__ constexpr int gemm_smem_bytes(int BN) { return gemm_stages(BN) * gemm_stage_bytes(BN) + 1024 + 256; }

namespace ptx {
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait: false when the barrier did not flip within GEMM_WAIT_CYCLES.
__device__ __forceinline__ bool mbar_wait_thread(uint32_t bar, uint32_t parity) {
  for (int i = 0; i < 128; ++i)
    if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  while (true) {
    if (mbar_try_wait(bar, parity)) return true;
    if (clock64() - t0 > GEMM_WAIT_CYCLES) return false;
  }
}
// The same for a whole converged warp; the outcome is made uniform so that no lane leaves a
// .sync.aligned section alone.
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity) {
  return __all_sync(0xffffffffu, mbar_wait_thread(bar, parity)) != 0;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t addr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(addr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t da, uint64_t db, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}"
      ::"r"(d_tmem), "l"(da), "l"(db), "r"(idesc), "r"(acc), "r"(0u) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t addr, uint32_t v[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
      : "r"(addr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
}  // namespace ptx

// Shared-memory matrix descriptor of a K-major tile stored with the 128-byte swizzle: rows are 128 B
// apart, groups of 8 rows 1024 B apart (stride byte offset), descriptor version 1, layout type 2.
__device__ __forceinline__ uint64_t umma_desc_sw128(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr >> 4) & 0x3FFF);
  d |= (uint64_t)1 << 16;                 // leading byte offset (unused with swizzle), 16 B units
  d |= (uint64_t)(1024 >> 4) << 32;       // stride byte offset
  d |= (uint64_t)1 << 46;                 // version
  d |= (uint64_t)2 << 61;                 // SWIZZLE_128B
  return d;
}

// Instruction descriptor: fp32 accumulator, bf16 A and B, both K-major, M = 128, N = BN.
__host__ __device__ constexpr uint32_t umma_idesc_bf16(int BN) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(GEMM_BM >> 4) << 24);
}

struct GemmArgs {
  int M, N, K;
  const float* bias;    // [N] or null
  void* out;            // EPI_STORE/GELU: bf16 [M, ldo]; EPI_RESID: fp32 [M, ldo] updated in place; EPI_F32: fp32
  int ldo;
  int* status;          // device word; set to TSDP_ERR_TIMEOUT (5) when a wait expires
};

template <int EPI>
__device__ __forceinline__ void epilogue_store16(const GemmArgs& g, int row, int col, const uint32_t v[16]) {
  float f[16];
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    f[i] = __uint_as_float(v[i]);
    if (g.bias) f[i] += __ldg(g.bias + col + i);
    if (EPI == EPI_GELU) f[i] = gelu_tanh(f[i]);
  }
  if (EPI == EPI_STORE || EPI == EPI_GELU) {
    __nv_bfloat16* o = reinterpret_cast<__nv_bfloat16*>(g.out) + (size_t)row * g.ldo + col;
    uint4 p[2];
    uint32_t* pw = reinterpret_cast<uint32_t*>(p);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      __nv_bfloat162 h2 = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
      pw[i] = *reinterpret_cast<uint32_t*>(&h2);
    }
    reinterpret_cast<uint4*>(o)[0] = p[0];
    reinterpret_cast<uint4*>(o)[1] = p[1];
  } else {
    float* o = reinterpret_cast<float*>(g.out) + (size_t)row * g.ldo + col;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      float4 r = make_float4(f[4 * i], f[4 * i + 1], f[4 * i + 2], f[4 * i + 3]);
      if (EPI == EPI_RESID) {
        const float4 h = reinterpret_cast<const float4*>(o)[i];
        r.x += h.x; r.y += h.y; r.z += h.z; r.w += h.w;
      }
      reinterpret_cast<float4*>(o)[i] = r;
    }
  }
}

template <int BN, int EPI>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
gemm_tcgen05_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, GemmArgs g) {
  constexpr int STAGES = gemm_stages(BN);
  constexpr int A_BYTES = GEMM_BM * GEMM_BK * 2;
  constexpr int STAGE_BYTES = gemm_stage_bytes(BN);
  constexpr uint32_t TMEM_COLS = (2 * BN < 32) ? 32 : 2 * BN;
  constexpr uint32_t IDESC = umma_idesc_bf16(BN);
  static_assert(BN == 32 || BN == 64 || BN == 128 || BN == 256, "BN");

  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t bar0 = base + STAGES * STAGE_BYTES;       // full[STAGES], empty[STAGES], tfull[2], tempty[2]
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (STAGES + s); };
  auto tfull_bar = [&](int s) { return bar0 + 8u * (2 * STAGES + s); };
  auto tempty_bar = [&](int s) { return bar0 + 8u * (2 * STAGES + 2 + s); };
  const uint32_t tmem_slot = bar0 + 8u * (2 * STAGES + 4);
  volatile uint32_t* tmem_slot_ptr =
      reinterpret_cast<volatile uint32_t*>(smem_raw + (tmem_slot - ptx::smem_u32(smem_raw)));

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tiles_m = (g.M + GEMM_BM - 1) / GEMM_BM;
  const int tiles_n = g.N / BN;
  const int n_tiles = tiles_m * tiles_n;
  const int kblocks = g.K / GEMM_BK;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { ptx::mbar_init(full_bar(s), 1); ptx::mbar_init(empty_bar(s), 1); }
    for (int s = 0; s < 2; ++s) { ptx::mbar_init(tfull_bar(s), 1); ptx::mbar_init(tempty_bar(s), GEMM_EPI_WARPS); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    ptx::tmem_alloc(tmem_slot, TMEM_COLS);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot_ptr;
  bool ok = true;

  if (warp == 0) {
    if (lane == 0) {
      int stage = 0; uint32_t phase = 0;
      for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
        const int tm = tile / tiles_n, tn = tile % tiles_n;
        for (int kb = 0; kb < kblocks; ++kb) {
          if (!ptx::mbar_wait_thread(empty_bar(stage), phase ^ 1u)) { ok = false; break; }
          ptx::mbar_expect_tx(full_bar(stage), STAGE_BYTES);
          const uint32_t sa = base + stage * STAGE_BYTES;
          ptx::tma_load_2d(sa, &tmA, kb * GEMM_BK, tm * GEMM_BM, full_bar(stage));
          ptx::tma_load_2d(sa + A_BYTES, &tmB, kb * GEMM_BK, tn * BN, full_bar(stage));
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      int stage = 0; uint32_t phase = 0; int it = 0;
      for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x, ++it) {
        const int as = it & 1; const uint32_t aphase = (it >> 1) & 1;
        if (!ptx::mbar_wait_thread(tempty_bar(as), aphase ^ 1u)) { ok = false; break; }
        ptx::tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(as * BN);
        for (int kb = 0; kb < kblocks; ++kb) {
          if (!ptx::mbar_wait_thread(full_bar(stage), phase)) { ok = false; break; }
          ptx::tc_fence_after();
          const uint32_t sa = base + stage * STAGE_BYTES;
          const uint64_t da = umma_desc_sw128(sa), db = umma_desc_sw128(sa + A_BYTES);
#pragma unroll
          for (int k = 0; k < GEMM_BK / 16; ++k)
            ptx::tc_mma_bf16(d_tmem, da + (uint64_t)(2 * k), db + (uint64_t)(2 * k), IDESC, (kb | k) ? 1u : 0u);
          ptx::tc_commit(empty_bar(stage));
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        ptx::tc_commit(tfull_bar(as));
      }
    }
  } else {
    const int ew = warp - 2;
    const int quad = warp & 3;               // TMEM lanes [32*quad, 32*quad+32) are this warp's
    const int half = ew >> 2;                // which half of the tile's columns
    constexpr int COLS = BN / 2;
    int it = 0;
    for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x, ++it) {
      const int tm = tile / tiles_n, tn = tile % tiles_n;
      const int as = it & 1; const uint32_t aphase = (it >> 1) & 1;
      if (!ptx::mbar_wait_warp(tfull_bar(as), aphase)) { ok = false; break; }
      ptx::tc_fence_after();
      const int row = tm * GEMM_BM + quad * 32 + lane;
      const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(as * BN + half * COLS);
#pragma unroll 1
      for (int c = 0; c < COLS; c += 16) {
        uint32_t v[16];
        ptx::tmem_ld16(taddr + (uint32_t)c, v);
        ptx::tmem_ld_wait();
        if (row < g.M) epilogue_store16<EPI>(g, row, tn * BN + half * COLS + c, v);
      }
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(tempty_bar(as));
    }
  }
  if (!ok) {
    atomicExch(g.status, 5);
    // let copies that are still in flight land before the shared memory is given back
    const long long t0 = clock64();
    while (clock64() - t0 < 400000ll) { }
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  if (warp == 1) ptx::tmem_dealloc(tmem_base, TMEM_COLS);
}

}  // namespace tsdp
