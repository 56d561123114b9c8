// bf16 GEMM for sm_100a:  C[M,N] = A[M,K] * W[N,K]^T (+ bias, activation, residual), fp32 accumulate.
//
// This is the dense contraction of the verification forward (Sec. 3.2, "Verification of Speculative
// Drafts": the frozen base model sees every candidate of the set C in one batched pass): every linear layer of the
// base transformer applied to all (K+1)*B candidate latents at once.
//
// Structure (one persistent CTA per SM, 128 x BN output tiles, BK = 64):
//   warp 0      TMA producer: cp.async.bulk.tensor 2-D tiles of A and W (both K-major, 128-byte
//               swizzle) into a ring of shared-memory stages, completion on mbarriers.
//   warp 1      MMA issuer: one elected thread issues tcgen05.mma (128 x BN x 16, kind::f16, bf16
//               inputs) into one of two TMEM accumulator buffers; tcgen05.commit releases smem
//               stages and publishes finished accumulators.
//   warps 2..9  epilogue: tcgen05.ld the accumulator (each warp owns one 32-lane TMEM quadrant and
//               half of the columns), fuse bias / GELU, and hand the tile back through shared
//               memory: 128-row x 128-byte chunks in the 128-byte-swizzled layout, written to global
//               memory by TMA (cp.async.bulk.tensor store; for the fp32 residual stream the TMA
//               reduce-add, so the residual is never read into the SM).  Tiles narrower than 128
//               columns store straight from registers.  The second accumulator buffer lets the
//               next tile's MMAs overlap this tile's epilogue.
// Every mbarrier wait is bounded: on expiry the kernel records TSDP_ERR_TIMEOUT in `status`, drains,
// frees its TMEM and returns.  This form is launched without clusters; the CTA-pair form further down runs in clusters
// of two.  No operand load is multicast in either: every CTA fetches its own tiles.
#pragma once
#include <cuda.h>
#include "common.cuh"

namespace tsdp {

// EPI_GATE: fp32 out += gate[tau(row), col] * (acc + bias), the gated residual of an adaptive-LayerNorm block.
// EPI_SILU: fp32 store of SiLU(acc + bias); CUDA-core GEMM only (conditioning tables built at load).
// EPI_MISH: as EPI_SILU with Mish.
// EPI_ATTN: the QKV projection with the self-attention fused into its epilogue (tensor-core kernel only, BN = 192):
//           output tile column block tn = head tn's [Q | K | V] (64 columns each, weights stored in that order), a
//           128-row tile = 8 candidates of 16 tokens; the epilogue runs the 16-token attention of each (candidate,
//           head) from shared memory and writes only the attention output, bf16 [M, d] at columns [64 tn, +64).
enum { EPI_STORE = 0, EPI_GELU = 1, EPI_RESID = 2, EPI_F32 = 3, EPI_GATE = 4, EPI_SILU = 5, EPI_MISH = 6, EPI_ATTN = 7 };

constexpr int GEMM_BM = 128;
constexpr int GEMM_BK = 64;
constexpr int GEMM_THREADS = 320;
constexpr int GEMM_EPI_WARPS = 8;
constexpr long long GEMM_WAIT_CYCLES = 2000000000ll;   // about one second of SM clock

__host__ __device__ constexpr int gemm_stages(int BN) { return BN >= 192 ? 4 : (BN >= 128 ? 6 : 8); }
__host__ __device__ constexpr int gemm_stage_bytes(int BN) { return GEMM_BM * GEMM_BK * 2 + BN * GEMM_BK * 2; }
constexpr int GEMM_STAGING_BYTES = 2 * 128 * 128;   // one 128-row x 128-byte chunk per column half
constexpr int GEMM_ATTN_BN = 192;                   // [Q | K | V] of one 64-wide head
constexpr int GEMM_ATTN_P = 64 + 8;                 // row pitch (elements) of the staged Q / K / V tiles
constexpr int GEMM_ATTN_STAGING_BYTES = 8 * 3 * 16 * GEMM_ATTN_P * 2;   // 8 candidates x {Q, K, V} x 16 rows
__host__ __device__ constexpr bool gemm_tma_epilogue(int BN) { return BN >= 128 && BN != GEMM_ATTN_BN; }
__host__ __device__ constexpr int gemm_epi_smem_bytes(int BN) {
  return BN == GEMM_ATTN_BN ? GEMM_ATTN_STAGING_BYTES : (gemm_tma_epilogue(BN) ? GEMM_STAGING_BYTES : 0);
}
// The tile's bias values, staged once per tile (one tile ahead of their use) so that no epilogue warp waits on a
// global load between its tensor-memory reads: 128 floats per column half, or one copy of the head's 192 per
// row quadrant in the fused-attention kernel (whose warps only synchronise quadrant by quadrant).
__host__ __device__ constexpr int gemm_bias_smem_bytes(int BN) { return BN == GEMM_ATTN_BN ? 4 * GEMM_ATTN_BN * 4 : 2 * 128 * 4; }
__host__ __device__ constexpr int gemm_smem_bytes(int BN) {
  return gemm_stages(BN) * gemm_stage_bytes(BN) + gemm_epi_smem_bytes(BN) + 1024 + 256 + gemm_bias_smem_bytes(BN);
}
// CTA-pair form (CG = 2, tcgen05 cta_group::2): a 256 x BN tile on two SMs.  Each CTA stages its own 128 rows of A and
// HALF of the W tile, so a stage is smaller and the ring deeper.
// The smaller stages also leave room for two staging chunks per column half, so that the epilogue does not have to
// wait for its previous TMA store (which queues behind the operand loads) before it fills the next chunk.
__host__ __device__ constexpr int gemm_stage_bytes_cg(int BN, int CG) { return GEMM_BM * GEMM_BK * 2 + (BN / CG) * GEMM_BK * 2; }
__host__ __device__ constexpr int gemm_stages_cg(int BN, int CG) { return CG == 2 ? (BN == GEMM_ATTN_BN ? 6 : 5) : gemm_stages(BN); }
__host__ __device__ constexpr int gemm_staging_bufs(int CG) { return CG == 2 ? 2 : 1; }      // per column half
__host__ __device__ constexpr int gemm_epi_smem_bytes_cg(int BN, int CG) {
  return gemm_tma_epilogue(BN) ? GEMM_STAGING_BYTES * gemm_staging_bufs(CG) : gemm_epi_smem_bytes(BN);
}
__host__ __device__ constexpr int gemm_smem_bytes_cg(int BN, int CG) {
  return gemm_stages_cg(BN, CG) * gemm_stage_bytes_cg(BN, CG) + gemm_epi_smem_bytes_cg(BN, CG) + 1024 + 256 + gemm_bias_smem_bytes(BN);
}

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
// Bounded wait: false when the barrier did not flip within `limit` SM clock cycles.
__device__ __forceinline__ bool mbar_wait_thread(uint32_t bar, uint32_t parity, long long limit = GEMM_WAIT_CYCLES) {
  for (int i = 0; i < 128; ++i)
    if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  while (true) {
    if (mbar_try_wait(bar, parity)) return true;
    if (clock64() - t0 > limit) return false;
  }
}
// The same for a whole converged warp; the outcome is made uniform so that no lane leaves a
// .sync.aligned section alone.
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, long long limit = GEMM_WAIT_CYCLES) {
  return __all_sync(0xffffffffu, mbar_wait_thread(bar, parity, limit)) != 0;
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
// ---- CTA-pair (cta_group::2) forms.  The two CTAs of a cluster of 2 act as one tensor-core unit: the leader (cluster
// rank 0) issues the MMAs, which read A from each CTA's own shared memory and one half of the B tile from each.
__device__ __forceinline__ uint32_t cluster_rank() { uint32_t r; asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r)); return r; }
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// shared::cluster address of the same shared-memory location in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t mapa_rank(uint32_t addr, uint32_t rank) {
  uint32_t r; asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank)); return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// TMA load whose completion is counted on a barrier that may live in the peer CTA (no multicast: each CTA fetches its own tiles)
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar_cluster_addr) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar_cluster_addr) : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t dst_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t addr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(addr), "r"(ncols) : "memory");
}
// arrive on the barrier at this shared-memory offset in BOTH CTAs of the pair once the MMAs issued so far are done
__device__ __forceinline__ void tc_commit_pair(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"((uint16_t)3) : "memory");
}
__device__ __forceinline__ void tc_mma_bf16_pair(uint32_t d_tmem, uint64_t da, uint64_t db, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(da), "l"(db), "r"(idesc), "r"(acc) : "memory");
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
__device__ __forceinline__ void tmem_ld32(uint32_t addr, uint32_t v[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
      "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
        "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
        "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(addr) : "memory");
}
// TMA store / reduce-add of one shared-memory box into a tiled global tensor (bulk async-group).
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, int x, int y, uint32_t src) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
               ::"l"(map), "r"(x), "r"(y), "r"(src) : "memory");
}
__device__ __forceinline__ void tma_reduce_add_2d(const CUtensorMap* map, int x, int y, uint32_t src) {
  asm volatile("cp.reduce.async.bulk.tensor.2d.global.shared::cta.add.tile.bulk_group [%0, {%1, %2}], [%3];"
               ::"l"(map), "r"(x), "r"(y), "r"(src) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read0() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read1() { asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void named_bar_sync(int id, int nthreads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}
// Barrier over `nthreads` threads that also ANDs a predicate across them.
__device__ __forceinline__ bool named_bar_and(int id, int nthreads, bool pred) {
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.u32 q, %1, 0;\n\t"
      "bar.red.and.pred p, %2, %3, q;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(r) : "r"(pred ? 1u : 0u), "r"(id), "r"(nthreads) : "memory");
  return r != 0;
}
__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ float tanh_fast(float x) {
  float y;
  asm("tanh.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// GELU (tanh form) on the hardware tanh, every operation spelled out so that each place that uses it --
// both GEMM epilogues and the cluster kernel -- produces the same bits whatever the compiler would contract.
__device__ __forceinline__ float gelu_fast(float x) {
  const float x3 = __fmul_rn(__fmul_rn(x, x), x);
  const float t = tanh_fast(__fmul_rn(0.7978845608028654f, __fmaf_rn(0.044715f, x3, x)));
  return __fmul_rn(__fmul_rn(0.5f, x), __fadd_rn(1.0f, t));
}
// Two values at a time on the packed fp32 pipe: every operation is the per-component round-to-nearest one of
// gelu_fast, so the bits are the same.
__device__ __forceinline__ float2 gelu_fast2(float2 x) {
  const float2 x3 = __fmul2_rn(__fmul2_rn(x, x), x);
  const float2 u = __fmul2_rn(make_float2(0.7978845608028654f, 0.7978845608028654f),
                              __ffma2_rn(make_float2(0.044715f, 0.044715f), x3, x));
  const float2 t = make_float2(tanh_fast(u.x), tanh_fast(u.y));
  return __fmul2_rn(__fmul2_rn(make_float2(0.5f, 0.5f), x), __fadd2_rn(make_float2(1.0f, 1.0f), t));
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
__host__ __device__ constexpr uint32_t umma_idesc_bf16(int BN, int M = GEMM_BM) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 h2 = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&h2);
}

struct GemmArgs {
  int M, N, K;
  const float* bias;    // [N] or null
  void* out;            // EPI_STORE/GELU: bf16 [M, ldo]; EPI_RESID: fp32 [M, ldo] updated in place; EPI_F32: fp32
  int ldo;
  int* status;          // device word; set to TSDP_ERR_TIMEOUT (5) when a wait expires
  // EPI_GATE only: gate vectors [Tsteps, gate_ld] (this layer's gate starts at column 0 of the pointer) and
  // the map from a token row to its timestep: row -> candidate n = row / H -> (b = n / C, c = n % C),
  // tau = clamp(t[b] - koff - c)
  const float* gate;
  int gate_ld;
  const int* t;
  int C, koff, H, Tsteps;
  int lda;              // row pitch of A in elements (CUDA-core GEMM; the tensor-core one has it in its tensor map)
  // Kernel-5 convolution over a zero-padded channels-last tensor [rows, conv_c] (0: plain GEMM): logical A row m
  // is the 5 conv_c elements starting at tensor row m, so k-block kb is tensor rows m + tap, columns
  // [c0, c0 + 64) with tap = (64 kb) / conv_c, c0 = (64 kb) % conv_c; conv_c is a multiple of 64.
  int conv_c;
  // Rows that really exist when the forward runs on a compacted candidate list: min(M, *live.n * live.mul + live.add)
  // (live.n null: M).  The tensor maps keep their full extent; tiles beyond the live rows are simply not visited.
  LiveRows live;
  const int* list;      // EPI_GATE with a compacted list: candidate n of a row is (list[n] >> 6, list[n] & 63)
  long long wait_cycles;  // limit of every mbarrier wait in SM clock cycles (0: GEMM_WAIT_CYCLES, about a second)
  // Test of the time-out path (host-armed, one launch): CTA 0's producer leaves out the operand loads of its very
  // first pipeline stage, so the waits that depend on that stage run out, the CTA reports TSDP_ERR_TIMEOUT through
  // `status`, drains and returns; every other CTA finishes its tiles as usual.
  int withhold_first_stage;
  int causal;           // EPI_ATTN: causal mask of the fused 16-token self-attention
  // Split reduction (narrow tiles with the plain-store epilogue, EPI_F32 only; 0 or 1: off): the k-blocks of every
  // tile are cut into `ksplit` contiguous parts, each a work unit of its own whose partial sums go to the buffer
  // out + part * split_stride (elements); the bias goes into part 0.  The consumer adds the parts in a fixed order,
  // so the result does not depend on which CTA ran which part.  For deep reductions over few rows (the convolutions
  // of a small batch), where the tiles alone occupy a fraction of the SMs.
  int ksplit;
  long long split_stride;
};

__device__ __forceinline__ const float* gate_row(const GemmArgs& g, int row) {
  const int n = row / g.H;
  int tau = g.list ? g.t[g.list[n] >> 6] - g.koff - (g.list[n] & 63) : g.t[n / g.C] - g.koff - (n % g.C);
  tau = max(0, min(g.Tsteps - 1, tau));
  return g.gate + (size_t)tau * g.gate_ld;
}

// `bias16`: the 16 bias values of these columns (fetched by the caller before it waited for the accumulator).
template <int EPI>
__device__ __forceinline__ void epilogue_store16(const GemmArgs& g, int row, int col, const uint32_t v[16], const float* bias16,
                                                 bool add_bias = true, size_t out_off = 0) {
  float f[16];
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    f[i] = __uint_as_float(v[i]);
    if (g.bias && add_bias) f[i] += bias16[i];
    if (EPI == EPI_GELU) f[i] = ptx::gelu_fast(f[i]);
  }
  if (EPI == EPI_GATE) {
    const float* gp = gate_row(g, row) + col;
#pragma unroll
    for (int i = 0; i < 16; ++i) f[i] *= __ldg(gp + i);
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
    float* o = reinterpret_cast<float*>(g.out) + out_off + (size_t)row * g.ldo + col;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      float4 r = make_float4(f[4 * i], f[4 * i + 1], f[4 * i + 2], f[4 * i + 3]);
      if (EPI == EPI_RESID || EPI == EPI_GATE) {
        const float4 h = reinterpret_cast<const float4*>(o)[i];
        r.x += h.x; r.y += h.y; r.z += h.z; r.w += h.w;
      }
      reinterpret_cast<float4*>(o)[i] = r;
    }
  }
}

// CG = 1: one CTA per 128 x BN tile.  CG = 2: launched in clusters of two CTAs that share a 256 x BN tile (cta_group::2):
// CTA `rank` owns rows [128 rank, +128) of the tile and stages rows [rank BN/2, +BN/2) of the W tile; the leader's MMA
// warp issues for both; stage and accumulator hand-over barriers are signalled in both CTAs by multicast commits, the
// stage-full and accumulator-empty barriers live in the leader and are signalled from both CTAs.  Per flop each SM
// pulls a third fewer operand bytes from the L2, which is what bounds the 128 x 256 form at K = 512.
template <int BN, int EPI, int CG = 1>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
gemm_tcgen05_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                    const __grid_constant__ CUtensorMap tmC, GemmArgs g) {
  constexpr int STAGES = gemm_stages_cg(BN, CG);
  constexpr int A_BYTES = GEMM_BM * GEMM_BK * 2;
  constexpr int B_ROWS = BN / CG;                      // rows of the W tile this CTA stages
  constexpr int STAGE_BYTES = gemm_stage_bytes_cg(BN, CG);
  static_assert(CG == 1 || CG == 2, "CG");
  static_assert(CG == 1 || BN == 256 || BN == GEMM_ATTN_BN, "pair form: wide tiles only");
  constexpr int ACC = BN == GEMM_ATTN_BN ? 256 : BN;          // column distance of the two accumulator buffers
  constexpr uint32_t TMEM_COLS = (2 * ACC < 32) ? 32 : 2 * ACC;  // a power of two
  constexpr uint32_t IDESC = umma_idesc_bf16(BN, GEMM_BM * CG);
  static_assert(BN == 32 || BN == 64 || BN == 128 || BN == 256 || BN == GEMM_ATTN_BN, "BN");
  static_assert((EPI == EPI_ATTN) == (BN == GEMM_ATTN_BN), "the fused attention epilogue has its own tile width");

  extern __shared__ uint8_t smem_raw[];
  pdl_trigger();
  const uint32_t base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
  constexpr bool TMA_EPI = gemm_tma_epilogue(BN);
  const uint32_t staging = base + STAGES * STAGE_BYTES;    // 1024-byte aligned: every stage is a multiple of 1 KB
  const uint32_t bar0 = staging + gemm_epi_smem_bytes_cg(BN, CG);   // full[STAGES], empty[STAGES], tfull[2], tempty[2]
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (STAGES + s); };
  auto tfull_bar = [&](int s) { return bar0 + 8u * (2 * STAGES + s); };
  auto tempty_bar = [&](int s) { return bar0 + 8u * (2 * STAGES + 2 + s); };
  const uint32_t tmem_slot = bar0 + 8u * (2 * STAGES + 4);
  volatile uint32_t* tmem_slot_ptr =
      reinterpret_cast<volatile uint32_t*>(smem_raw + (tmem_slot - ptx::smem_u32(smem_raw)));
  float* sbias = reinterpret_cast<float*>(smem_raw + (bar0 + 256u - ptx::smem_u32(smem_raw)));    // behind the barriers

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tiles_n = g.N / BN;
  const int kblocks = g.K / GEMM_BK;
  const uint32_t rank = CG == 2 ? ptx::cluster_rank() : 0u;     // 0: the pair's leader

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { ptx::mbar_init(full_bar(s), 1); ptx::mbar_init(empty_bar(s), 1); }
    for (int s = 0; s < 2; ++s) { ptx::mbar_init(tfull_bar(s), 1); ptx::mbar_init(tempty_bar(s), GEMM_EPI_WARPS * CG); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    if (CG == 2) { ptx::tmem_alloc_pair(tmem_slot, TMEM_COLS); ptx::tmem_relinquish_pair(); }
    else { ptx::tmem_alloc(tmem_slot, TMEM_COLS); ptx::tmem_relinquish(); }
  }
  ptx::tc_fence_before();
  __syncthreads();
  if (CG == 2) ptx::cluster_sync_all();      // the peer's barriers exist before anything is signalled across the pair
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot_ptr;
  bool ok = true;
  const long long wlim = g.wait_cycles > 0 ? g.wait_cycles : GEMM_WAIT_CYCLES;
  pdl_wait();      // operands, bias, the output and the live-row count belong to earlier kernels of the stream
  const int M = live_rows(g.live, g.M);
  const int tiles_m = (M + GEMM_BM * CG - 1) / (GEMM_BM * CG);     // tiles of 128 CG rows
  const int S = g.ksplit > 1 ? g.ksplit : 1;                       // parts of the reduction (plain-store epilogue only)
  const int n_tiles = tiles_m * tiles_n * S;                       // work units: (tile, part), part fastest
  const int tile0 = blockIdx.x / CG, tile_step = gridDim.x / CG;      // both CTAs of a pair walk the same tiles
  // an epilogue warp hands accumulator buffer `as` back: the barrier that the MMA warp waits on lives in the leader
  auto release_acc = [&](int as) {
    if (CG == 2 && rank != 0) ptx::mbar_arrive_cluster(ptx::mapa_rank(tempty_bar(as), 0));
    else ptx::mbar_arrive(tempty_bar(as));
  };

  if (warp == 0) {
    if (lane == 0) {
      int stage = 0; uint32_t phase = 0;
      for (int unit = tile0; unit < n_tiles && ok; unit += tile_step) {
        const int tile = unit / S, part = unit - tile * S;
        const int tm = (tile / tiles_n) * CG + (int)rank, tn = tile % tiles_n;
        const int kb0 = part * kblocks / S, kb1 = (part + 1) * kblocks / S;
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!ptx::mbar_wait_thread(empty_bar(stage), phase ^ 1u, wlim)) { ok = false; break; }
          if (!(g.withhold_first_stage && blockIdx.x == 0 && unit == 0 && kb == 0)) {
            const uint32_t sa = base + stage * STAGE_BYTES;
            const int kcol = kb * GEMM_BK;
            const int ax = g.conv_c ? kcol % g.conv_c : kcol, ay = tm * GEMM_BM + (g.conv_c ? kcol / g.conv_c : 0);
            if (CG == 2) {
              // the leader's barrier counts the bytes of both CTAs' loads of this stage
              if (rank == 0) ptx::mbar_expect_tx(full_bar(stage), STAGE_BYTES * 2);
              const uint32_t fb = ptx::mapa_rank(full_bar(stage), 0);
              ptx::tma_load_2d_pair(sa, &tmA, ax, ay, fb);
              ptx::tma_load_2d_pair(sa + A_BYTES, &tmB, kb * GEMM_BK, tn * BN + (int)rank * B_ROWS, fb);
            } else {
              ptx::mbar_expect_tx(full_bar(stage), STAGE_BYTES);
              ptx::tma_load_2d(sa, &tmA, ax, ay, full_bar(stage));
              ptx::tma_load_2d(sa + A_BYTES, &tmB, kb * GEMM_BK, tn * BN, full_bar(stage));
            }
          }
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && rank == 0) {      // in a pair only the leader issues
      int stage = 0; uint32_t phase = 0; int it = 0;
      for (int unit = tile0; unit < n_tiles && ok; unit += tile_step, ++it) {
        const int part = unit % S;
        const int kb0 = part * kblocks / S, kb1 = (part + 1) * kblocks / S;
        const int as = it & 1; const uint32_t aphase = (it >> 1) & 1;
        if (!ptx::mbar_wait_thread(tempty_bar(as), aphase ^ 1u, wlim)) { ok = false; break; }
        ptx::tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(as * ACC);
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!ptx::mbar_wait_thread(full_bar(stage), phase, wlim)) { ok = false; break; }
          ptx::tc_fence_after();
          const uint32_t sa = base + stage * STAGE_BYTES;
          const uint64_t da = umma_desc_sw128(sa), db = umma_desc_sw128(sa + A_BYTES);
#pragma unroll
          for (int k = 0; k < GEMM_BK / 16; ++k) {
            if (CG == 2) ptx::tc_mma_bf16_pair(d_tmem, da + (uint64_t)(2 * k), db + (uint64_t)(2 * k), IDESC, (kb > kb0 || k) ? 1u : 0u);
            else ptx::tc_mma_bf16(d_tmem, da + (uint64_t)(2 * k), db + (uint64_t)(2 * k), IDESC, (kb > kb0 || k) ? 1u : 0u);
          }
          if (CG == 2) ptx::tc_commit_pair(empty_bar(stage)); else ptx::tc_commit(empty_bar(stage));
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        if (CG == 2) ptx::tc_commit_pair(tfull_bar(as)); else ptx::tc_commit(tfull_bar(as));
      }
    }
  } else {
    const int ew = warp - 2;
    const int quad = warp & 3;               // TMEM lanes [32*quad, 32*quad+32) are this warp's
    const int half = ew >> 2;                // which half of the tile's columns
    constexpr int COLS = BN / 2;
    int it = 0;
    if constexpr (EPI == EPI_ATTN) {
      // Rows 32 quad .. +31 of the tile are two candidates (16 tokens each); the two warps of a quadrant each bring
      // half of the 192 columns of those rows from tensor memory to shared memory (bias added, bf16), then each runs
      // the attention of one of the two candidates.  Only the two warps of a quadrant ever touch its staging area.
      constexpr int P = GEMM_ATTN_P;
      __nv_bfloat16* att = reinterpret_cast<__nv_bfloat16*>(smem_raw + (staging - ptx::smem_u32(smem_raw)));
      const int pair_bar = 1 + quad;
      const int r_tile = quad * 32 + lane;                    // this lane's row of the tile
      const int cand_l = r_tile >> 4, r_l = r_tile & 15;      // candidate (0..7) and token of that row
      const int cand_w = 2 * quad + half;                     // the candidate this warp attends for
      // the quadrant's copy of the head's bias: thread j of the pair brings values j, j + 64, j + 128, one tile ahead
      float* sb = sbias + quad * GEMM_ATTN_BN;
      const int bj = half * 32 + lane;
      float bnx[3] = {0.f, 0.f, 0.f};
      if (g.bias && tile0 < n_tiles) {
#pragma unroll
        for (int u = 0; u < 3; ++u) bnx[u] = __ldg(g.bias + (tile0 % tiles_n) * BN + bj + 64 * u);
      }
      for (int tile = tile0; tile < n_tiles; tile += tile_step, ++it) {
        const int tm = (tile / tiles_n) * CG + (int)rank, tn = tile % tiles_n;
        const int as = it & 1; const uint32_t aphase = (it >> 1) & 1;
        if (g.bias) {      // the previous tile's reads of `sb` lie before its staging barrier
#pragma unroll
          for (int u = 0; u < 3; ++u) sb[bj + 64 * u] = bnx[u];
          if (tile + tile_step < n_tiles) {
#pragma unroll
            for (int u = 0; u < 3; ++u) bnx[u] = __ldg(g.bias + ((tile + tile_step) % tiles_n) * BN + bj + 64 * u);
          }
        }
        // both warps of the quadrant agree on the outcome; the barrier also orders the previous tile's reads of the
        // staging area before this tile's writes, and publishes `sb`
        ok = ptx::named_bar_and(pair_bar, 64, ptx::mbar_wait_warp(tfull_bar(as), aphase, wlim));
        if (!ok) break;
        ptx::tc_fence_after();
        const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(as * ACC + half * 96);
#pragma unroll
        for (int part = 0; part < 3; ++part) {
          uint32_t v[32];
          ptx::tmem_ld32(taddr + (uint32_t)(part * 32), v);
          ptx::tmem_ld_wait();
          if (part == 2) {                                    // accumulator fully read: hand it back
            ptx::tc_fence_before();
            __syncwarp();
            if (lane == 0) release_acc(as);
          }
          const int col = half * 96 + part * 32;              // column inside the head's [Q | K | V]
          float f[32];
#pragma unroll
          for (int i = 0; i < 32; ++i) f[i] = __uint_as_float(v[i]);
          if (g.bias) {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              const float4 bb = reinterpret_cast<const float4*>(sb + col)[i];
              const float2 lo = __fadd2_rn(make_float2(f[4 * i], f[4 * i + 1]), make_float2(bb.x, bb.y));
              const float2 hi = __fadd2_rn(make_float2(f[4 * i + 2], f[4 * i + 3]), make_float2(bb.z, bb.w));
              f[4 * i] = lo.x; f[4 * i + 1] = lo.y; f[4 * i + 2] = hi.x; f[4 * i + 3] = hi.y;
            }
          }
          __nv_bfloat16* dst = att + ((size_t)(cand_l * 3 + (col >> 6)) * 16 + r_l) * P + (col & 63);
#pragma unroll
          for (int j = 0; j < 4; ++j)
            *reinterpret_cast<uint4*>(dst + 8 * j) =
                make_uint4(pack_bf16x2(f[8 * j], f[8 * j + 1]), pack_bf16x2(f[8 * j + 2], f[8 * j + 3]),
                           pack_bf16x2(f[8 * j + 4], f[8 * j + 5]), pack_bf16x2(f[8 * j + 6], f[8 * j + 7]));
        }
        ptx::named_bar_sync(pair_bar, 64);                    // the quadrant's Q, K, V tiles are complete
        __nv_bfloat16* sQ = att + (size_t)(cand_w * 3) * 16 * P;
        attn16_from_smem<64>(sQ, sQ + 16 * P, sQ + 32 * P, 16, g.causal, lane);
        __syncwarp();
        const int row0 = tm * GEMM_BM + cand_w * 16;
        __nv_bfloat16* o = reinterpret_cast<__nv_bfloat16*>(g.out) + (size_t)row0 * g.ldo + tn * 64;
#pragma unroll
        for (int i = lane; i < 16 * 8; i += 32) {
          const int r = i >> 3, v8 = i & 7;
          if (row0 + r < M)
            *reinterpret_cast<uint4*>(o + (size_t)r * g.ldo + v8 * 8) = *reinterpret_cast<const uint4*>(sQ + r * P + v8 * 8);
        }
      }
    } else if constexpr (TMA_EPI) {
      // Output element size, columns per 128-byte chunk, chunks per half tile.
      constexpr int ESZ = (EPI == EPI_STORE || EPI == EPI_GELU) ? 2 : 4;
      constexpr int CW = 128 / ESZ;
      constexpr int NCH = COLS / CW;
      // NB chunk buffers per column half, used in turn; a buffer is refilled once the store issued NB chunks ago has
      // read it (NB = 1: the previous one)
      constexpr int NB = gemm_staging_bufs(CG);
      const uint32_t stg0 = staging + (uint32_t)half * (uint32_t)(NB * (GEMM_STAGING_BYTES / 2));
      int chunk_no = 0;
      const int r = quad * 32 + lane;        // row of the tile this thread owns
      const uint32_t sw = (uint32_t)(r & 7);
      const bool issuer = (quad == 0 && lane == 0);
      const int bar_id = 1 + half;
      // this half's bias values of a tile: thread r brings value r, one tile ahead of its use
      float* sb = sbias + half * 128;
      const bool bias_lane = g.bias != nullptr && r < COLS;
      float bias_next = 0.f;
      if (bias_lane && tile0 < n_tiles) bias_next = __ldg(g.bias + (tile0 % tiles_n) * BN + half * COLS + r);
      constexpr int NPART = COLS / 32;       // 32-column parts of this half
      for (int tile = tile0; tile < n_tiles; tile += tile_step, ++it) {
        const int tm = (tile / tiles_n) * CG + (int)rank, tn = tile % tiles_n;
        const int as = it & 1; const uint32_t aphase = (it >> 1) & 1;
        if (bias_lane) {         // the previous tile's reads of `sb` lie before its last staging barrier
          sb[r] = bias_next;
          if (tile + tile_step < n_tiles) bias_next = __ldg(g.bias + ((tile + tile_step) % tiles_n) * BN + half * COLS + r);
        }
        // the row's gate values of the first part, in flight while the accumulator is awaited
        float4 gq[8];
        const float* gate_base = nullptr;
        if (EPI == EPI_GATE) {
          const int grow = min(tm * GEMM_BM + r, M - 1);       // rows past the live ones only reach rows nobody reads
          gate_base = gate_row(g, grow) + tn * BN + half * COLS;
#pragma unroll
          for (int i = 0; i < 8; ++i) gq[i] = __ldg(reinterpret_cast<const float4*>(gate_base) + i);
        }
        // all four warps of this half agree on the outcome, so none is left alone at a named barrier (which also
        // publishes `sb`)
        ok = ptx::named_bar_and(bar_id, 128, ptx::mbar_wait_warp(tfull_bar(as), aphase, wlim));
        if (!ok) break;
        ptx::tc_fence_after();
        const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(as * ACC + half * COLS);
#pragma unroll 1
        for (int ch = 0; ch < NCH; ++ch, ++chunk_no) {
          const uint32_t stg = stg0 + (uint32_t)(chunk_no % NB) * (uint32_t)(GEMM_STAGING_BYTES / 2);
          const uint32_t row_addr = stg + (uint32_t)r * 128u;
#pragma unroll
          for (int part = 0; part < CW / 32; ++part) {
            uint32_t v[32];
            const int col_t = ch * CW + part * 32;                 // column inside this half
            float4 gn[8];                                          // the next part's gate values: in flight during this one
            if (EPI == EPI_GATE && col_t + 32 < COLS) {
#pragma unroll
              for (int i = 0; i < 8; ++i) gn[i] = __ldg(reinterpret_cast<const float4*>(gate_base + col_t + 32) + i);
            }
            ptx::tmem_ld32(taddr + (uint32_t)col_t, v);
            ptx::tmem_ld_wait();
            if (ch == NCH - 1 && part == CW / 32 - 1) {            // accumulator fully read: hand it back
              ptx::tc_fence_before();
              __syncwarp();
              if (lane == 0) release_acc(as);
            }
            float2 f2[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) f2[i] = make_float2(__uint_as_float(v[2 * i]), __uint_as_float(v[2 * i + 1]));
            if (g.bias) {
#pragma unroll
              for (int i = 0; i < 8; ++i) {
                const float4 bb = reinterpret_cast<const float4*>(sb + col_t)[i];
                f2[2 * i] = __fadd2_rn(f2[2 * i], make_float2(bb.x, bb.y));
                f2[2 * i + 1] = __fadd2_rn(f2[2 * i + 1], make_float2(bb.z, bb.w));
              }
            }
            if (EPI == EPI_GELU) {
#pragma unroll
              for (int i = 0; i < 16; ++i) f2[i] = ptx::gelu_fast2(f2[i]);
            }
            if (EPI == EPI_GATE) {
#pragma unroll
              for (int i = 0; i < 8; ++i) {
                f2[2 * i] = __fmul2_rn(f2[2 * i], make_float2(gq[i].x, gq[i].y));
                f2[2 * i + 1] = __fmul2_rn(f2[2 * i + 1], make_float2(gq[i].z, gq[i].w));
              }
              if (col_t + 32 < COLS) {
#pragma unroll
                for (int i = 0; i < 8; ++i) gq[i] = gn[i];
              }
            }
            float f[32];
#pragma unroll
            for (int i = 0; i < 16; ++i) { f[2 * i] = f2[i].x; f[2 * i + 1] = f2[i].y; }
            if (part == 0) {   // the TMA store that last used this staging buffer must have read it
              if (issuer) { if (NB == 2) ptx::bulk_wait_read1(); else ptx::bulk_wait_read0(); }
              ptx::named_bar_sync(bar_id, 128);
            }
            if (ESZ == 2) {
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                const uint32_t c16 = (uint32_t)(part * 4 + j);
                ptx::st_shared_v4(row_addr + ((c16 ^ sw) << 4),
                                  pack_bf16x2(f[8 * j], f[8 * j + 1]), pack_bf16x2(f[8 * j + 2], f[8 * j + 3]),
                                  pack_bf16x2(f[8 * j + 4], f[8 * j + 5]), pack_bf16x2(f[8 * j + 6], f[8 * j + 7]));
              }
            } else {
#pragma unroll
              for (int j = 0; j < 8; ++j)
                ptx::st_shared_v4(row_addr + (((uint32_t)j ^ sw) << 4), __float_as_uint(f[4 * j]),
                                  __float_as_uint(f[4 * j + 1]), __float_as_uint(f[4 * j + 2]), __float_as_uint(f[4 * j + 3]));
            }
          }
          ptx::fence_async_smem();
          ptx::named_bar_sync(bar_id, 128);
          if (issuer) {
            const int x = tn * BN + half * COLS + ch * CW, y = tm * GEMM_BM;
            if (EPI == EPI_RESID || EPI == EPI_GATE) ptx::tma_reduce_add_2d(&tmC, x, y, stg);
            else ptx::tma_store_2d(&tmC, x, y, stg);
            ptx::bulk_commit();
          }
        }
      }
      if (issuer) ptx::bulk_wait_read0();
    } else {
      for (int unit = tile0; unit < n_tiles && ok; unit += tile_step, ++it) {
        const int tile = unit / S, part = unit - tile * S;
        const int tm = (tile / tiles_n) * CG + (int)rank, tn = tile % tiles_n;
        const int as = it & 1; const uint32_t aphase = (it >> 1) & 1;
        float bv[COLS];          // this half's bias values (narrow tiles: at most 32), fetched while the accumulator is awaited
        if (g.bias) {
#pragma unroll
          for (int i = 0; i < COLS / 4; ++i) {
            const float4 bb = __ldg(reinterpret_cast<const float4*>(g.bias + tn * BN + half * COLS) + i);
            bv[4 * i] = bb.x; bv[4 * i + 1] = bb.y; bv[4 * i + 2] = bb.z; bv[4 * i + 3] = bb.w;
          }
        }
        if (!ptx::mbar_wait_warp(tfull_bar(as), aphase, wlim)) { ok = false; break; }
        ptx::tc_fence_after();
        const int row = tm * GEMM_BM + quad * 32 + lane;
        const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(as * ACC + half * COLS);
#pragma unroll
        for (int c = 0; c < COLS; c += 16) {
          uint32_t v[16];
          ptx::tmem_ld16(taddr + (uint32_t)c, v);
          ptx::tmem_ld_wait();
          if (row < M) epilogue_store16<EPI>(g, row, tn * BN + half * COLS + c, v, bv + c, part == 0, (size_t)part * (size_t)g.split_stride);
        }
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) release_acc(as);
      }
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
  if (CG == 2) ptx::cluster_sync_all();      // neither CTA leaves while its peer may still signal or read it
  ptx::tc_fence_after();
  if (warp == 1) {
    if (CG == 2) ptx::tmem_dealloc_pair(tmem_base, TMEM_COLS);
    else ptx::tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

}  // namespace tsdp
