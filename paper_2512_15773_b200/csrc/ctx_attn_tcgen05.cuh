// Cross-attention of the action tokens to the context tokens of their request (adaptive-LayerNorm transformer,
// the VLA-scale action expert) on the 5th-generation tensor cores, for 64-wide heads and bf16 activations.
//
// One CTA per (group, head), where a group is the set of query rows that share one request's context: all
// candidates of a batch slot in the verification forward (up to (K+1) H rows), one candidate in a drafter forward.
// The head's keys K [Tc x 64] and values V [Tc x 64] (projected once per chunk) are fetched once by TMA; V is
// re-laid out in shared memory as V^T so that both products take K-major operands.  Then, per tile of 128 query rows:
//   TMA      Q tile [128 x 64] -> shared memory (double-buffered, the next tile is fetched during this one)
//   MMA 1    S = Q K^T      [128 x Tc], fp32, in tensor memory                      (tcgen05.mma, one issuing thread)
//   softmax  two threads per query row (warps w and w + 4 share tensor-memory lane quadrant w and split the Tc
//            columns): two passes over the scores straight from tensor memory (tcgen05.ld), row maximum and row sum
//            exchanged through shared memory, p = exp2((s - max) log2(e) / sqrt(dh)); P goes back INTO tensor memory
//            as packed bf16 pairs (tcgen05.st), each thread over the first half of the score columns it has just read
//   MMA 2    O = P V        [128 x 64], fp32: A operand from tensor memory, V^T from shared memory; O lands in
//            columns 192..255 (score columns that are dead by then, or beyond the scores)
//   epilogue the same two threads read half a row of O each, scale by 1 / row sum, store 64 bytes of bf16 each.
// No online softmax: all Tc <= 256 scores of a row are in tensor memory at once.  With P in tensor memory a CTA needs
// 256 columns of it and under 100 KB of shared memory, so two CTAs share an SM and one's products run under the
// other's softmax (within a CTA the four steps of a tile are strictly serial).  Rows past the group's end are
// computed on whatever the tile fetched (other rows of the buffer, or zeros past its end) and never stored.
// Every mbarrier wait is bounded; on expiry the CTA records TSDP_ERR_TIMEOUT (5) in `status`, frees its tensor
// memory and returns.
#pragma once
#include "common.cuh"
#include "gemm_tcgen05.cuh"

namespace tsdp {

namespace ptx {
__device__ __forceinline__ void tmem_st8(uint32_t addr, const uint32_t v[8]) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
               ::"r"(addr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]) : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
// D (tensor memory) (+)= A (tensor memory: lane = row, one 32-bit column = two consecutive k) x B (shared memory)
__device__ __forceinline__ void tc_mma_bf16_ta(uint32_t d_tmem, uint32_t a_tmem, uint64_t db, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, {%5, %5, %5, %5}, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(db), "r"(idesc), "r"(acc), "r"(0u) : "memory");
}
}  // namespace ptx

constexpr int CXT_THREADS = 288;                 // warps 0-7: softmax / epilogue (two threads per row), warp 8: TMA + MMA issue
constexpr int CXT_Q_BYTES = 128 * 128;           // one Q tile: 128 rows x 64 bf16
constexpr int CXT_OFF_K = 2 * CXT_Q_BYTES;       // keys [Tc x 64], up to 32 KB; the two Q buffers first hold the V staging tile
constexpr int CXT_OFF_VT = CXT_OFF_K + 256 * 128;        // V^T as Tc/64 atoms of [64 x 64]
constexpr int CXT_OFF_BAR = CXT_OFF_VT + 256 * 128;
constexpr int CXT_OFF_X = CXT_OFF_BAR + 128;              // row maxima and row sums of the two column halves: float [2][2][128]
constexpr int CXT_SMEM_BYTES = CXT_OFF_X + 2048 + 1024;   // + alignment slack
constexpr uint32_t CXT_TMEM_COLS = 256;          // scores [0, Tc); P over [0, Tc/4) and [Tc/2, 3Tc/4); O in [192, 256)
constexpr uint32_t CXT_O_COL = 192;

__global__ void __launch_bounds__(CXT_THREADS, 2)
cross_attn_ctx_tc_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmKV,
                         __nv_bfloat16* __restrict__ out, int kv_off, CandMap cm, int rows_per_slot, int d, int heads, int Tc,
                         const int* __restrict__ slot_start, int H, int* __restrict__ status) {
  extern __shared__ uint8_t cxt_raw[];
  pdl_trigger();
  const uint32_t base = (ptx::smem_u32(cxt_raw) + 1023u) & ~1023u;
  uint8_t* gbase = cxt_raw + (base - ptx::smem_u32(cxt_raw));
  const uint32_t sQ = base, sK = base + CXT_OFF_K, sVt = base + CXT_OFF_VT, bar0 = base + CXT_OFF_BAR;
  const uint32_t bar_kv = bar0, bar_q0 = bar0 + 8, bar_s = bar0 + 24, bar_p = bar0 + 32, bar_o = bar0 + 40, bar_or = bar0 + 48;
  const uint32_t tmem_slot = bar0 + 64;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    ptx::mbar_init(bar_kv, 1); ptx::mbar_init(bar_q0, 1); ptx::mbar_init(bar_q0 + 8, 1);
    ptx::mbar_init(bar_s, 1); ptx::mbar_init(bar_p, 256); ptx::mbar_init(bar_o, 1); ptx::mbar_init(bar_or, 256);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 8) { ptx::tmem_alloc(tmem_slot, CXT_TMEM_COLS); ptx::tmem_relinquish(); }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(gbase + CXT_OFF_BAR + 64);
  pdl_wait();

  // rows of this group (see cross_attn_ctx_mma_kernel: dense slots, compacted slots, or one list entry per group)
  int b = blockIdx.x / heads;
  const int hd = blockIdx.x % heads;
  long long row0 = (long long)b * rows_per_slot;
  int rows = rows_per_slot;
  bool live = true;
  if (slot_start != nullptr) {
    row0 = (long long)slot_start[b] * H;
    rows = (slot_start[b + 1] - slot_start[b]) * H;
    live = rows > 0;
  } else if (cm.list != nullptr) {
    live = b < cand_count(cm, (int)(gridDim.x / heads));
    if (live) b = cm.list[b] >> 6;
  }
  const int n_tiles = live ? (rows + 127) / 128 : 0;
  bool ok = true;
  const uint32_t kv_bytes = (uint32_t)Tc * 128u;

  if (n_tiles > 0) {
    // ---- keys and values (the values into the staging tile, which is the two Q buffers)
    if (warp == 8 && lane == 0) {
      const int y = item_of(cm.item, b) * Tc;
      ptx::mbar_expect_tx(bar_kv, 2 * kv_bytes);
      ptx::tma_load_2d(sK, &tmKV, kv_off + hd * 64, y, bar_kv);
      ptx::tma_load_2d(sQ, &tmKV, kv_off + d + hd * 64, y, bar_kv);
    }
    ok = ptx::mbar_wait_thread(bar_kv, 0);
    ok = __syncthreads_and(ok ? 1 : 0) != 0;
    if (ok) {
      // V [Tc x 64] (128-byte-swizzled rows, as TMA wrote it) -> V^T: atom a = key / 64 holds [64 dh-rows x 64 keys]
      const uint8_t* vs = gbase;
      uint8_t* vt = gbase + CXT_OFF_VT;
      for (int i = threadIdx.x; i < Tc * 8; i += CXT_THREADS) {
        const int r = i >> 3, ch = i & 7;                 // key r, 16-byte chunk ch = dh columns 8 ch .. 8 ch + 7
        const uint4 v = *reinterpret_cast<const uint4*>(vs + r * 128 + ((ch ^ (r & 7)) << 4));
        const unsigned short* e = reinterpret_cast<const unsigned short*>(&v);
        const int atom = r >> 6, kk = r & 63;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const int n = ch * 8 + j;
          *reinterpret_cast<unsigned short*>(vt + atom * 8192 + n * 128 + (((kk >> 3) ^ (n & 7)) << 4) + (kk & 7) * 2) = e[j];
        }
      }
      ptx::fence_async_smem();       // V^T is read by the tensor core, and the staging tile is about to be overwritten by TMA
    }
    __syncthreads();
    if (ok && warp == 8 && lane == 0) {                    // the first Q tile, now that the staging tile is free
      ptx::mbar_expect_tx(bar_q0, CXT_Q_BYTES);
      ptx::tma_load_2d(sQ, &tmQ, hd * 64, (int)row0, bar_q0);
    }
  }

  const int hc = Tc / 2;                                    // score columns per softmax thread; a multiple of 16
  if (ok && n_tiles > 0) {
    if (warp == 8) {
      if (lane == 0) {
        const uint32_t idesc1 = umma_idesc_bf16(Tc, 128), idesc2 = umma_idesc_bf16(64, 128);
        for (int i = 0; i < n_tiles; ++i) {
          const uint32_t qb = sQ + (uint32_t)(i & 1) * CXT_Q_BYTES;
          if (!ptx::mbar_wait_thread(bar_q0 + 8u * (i & 1), (uint32_t)((i >> 1) & 1))) { ok = false; break; }
          // the scores overwrite P and (for Tc > 192) O of the previous tile: its second product is ahead in the
          // tensor pipe, its O must have been read
          if (i > 0 && !ptx::mbar_wait_thread(bar_or, (uint32_t)((i - 1) & 1))) { ok = false; break; }
          ptx::tc_fence_after();
          const uint64_t da = umma_desc_sw128(qb), db = umma_desc_sw128(sK);
#pragma unroll
          for (int k = 0; k < 4; ++k) ptx::tc_mma_bf16(tmem_base, da + (uint64_t)(2 * k), db + (uint64_t)(2 * k), idesc1, k ? 1u : 0u);
          ptx::tc_commit(bar_s);
          if (i + 1 < n_tiles) {      // the other Q buffer was last read by the first product of tile i - 1: complete
            const uint32_t nb = bar_q0 + 8u * ((i + 1) & 1);
            ptx::mbar_expect_tx(nb, CXT_Q_BYTES);
            ptx::tma_load_2d(sQ + (uint32_t)((i + 1) & 1) * CXT_Q_BYTES, &tmQ, hd * 64, (int)row0 + (i + 1) * 128, nb);
          }
          if (!ptx::mbar_wait_thread(bar_p, (uint32_t)(i & 1))) { ok = false; break; }
          ptx::tc_fence_after();
          for (int j = 0; j < Tc / 16; ++j) {               // keys 16 j .. 16 j + 15: eight columns of P
            const int pc = 16 * j < hc ? 8 * j : hc + 8 * (j - hc / 16);
            const uint64_t vb = umma_desc_sw128(sVt + (uint32_t)(j >> 2) * 8192u) + (uint64_t)(2 * (j & 3));
            ptx::tc_mma_bf16_ta(tmem_base + CXT_O_COL, tmem_base + (uint32_t)pc, vb, idesc2, j ? 1u : 0u);
          }
          ptx::tc_commit(bar_o);
        }
      }
    } else {
      const int quad = warp & 3, half = warp >> 2;          // tensor-memory lane quadrant; which half of the columns
      const int r = quad * 32 + lane;                       // query row of the tile; tensor-memory lane
      const uint32_t t_s = tmem_base + ((uint32_t)(quad * 32) << 16);
      const float c = 1.4426950408889634f * 0.125f;         // log2(e) / sqrt(64)
      float* xmax = reinterpret_cast<float*>(gbase + CXT_OFF_X);       // [2][128]
      float* xsum = xmax + 256;                                       // [2][128]
      const int cbeg = half * hc, cend = cbeg + hc;
      const int pair_bar = 1 + quad;                                  // the two warps of a quadrant
      for (int i = 0; i < n_tiles; ++i) {
        ok = ptx::named_bar_and(pair_bar, 64, ptx::mbar_wait_warp(bar_s, (uint32_t)(i & 1)));
        if (!ok) break;
        ptx::tc_fence_after();
        float mx = -INFINITY;
        for (int c0 = cbeg; c0 < cend; c0 += 16) {
          uint32_t v[16];
          ptx::tmem_ld16(t_s + (uint32_t)c0, v);
          ptx::tmem_ld_wait();
#pragma unroll
          for (int j = 0; j < 16; ++j) mx = fmaxf(mx, __uint_as_float(v[j]));
        }
        xmax[half * 128 + r] = mx;
        ptx::named_bar_sync(pair_bar, 64);
        mx = fmaxf(mx, xmax[(half ^ 1) * 128 + r]);
        const float mc = mx * c;
        float sum = 0.f;
        for (int c0 = cbeg; c0 < cend; c0 += 16) {
          uint32_t v[16];
          ptx::tmem_ld16(t_s + (uint32_t)c0, v);
          ptx::tmem_ld_wait();
          uint32_t pk[8];
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const float p0 = exp2f(__fmaf_rn(__uint_as_float(v[2 * j]), c, -mc));
            const float p1 = exp2f(__fmaf_rn(__uint_as_float(v[2 * j + 1]), c, -mc));
            sum += p0 + p1;
            pk[j] = pack_bf16x2(p0, p1);
          }
          // keys c0 .. c0 + 15 of this row -> columns cbeg + (c0 - cbeg) / 2 .. + 7: behind this thread's own reads
          ptx::tmem_st8(t_s + (uint32_t)(cbeg + ((c0 - cbeg) >> 1)), pk);
        }
        xsum[half * 128 + r] = sum;
        ptx::tmem_st_wait();                                // P is in tensor memory
        ptx::tc_fence_before();                             // and the scores have been read
        ptx::mbar_arrive(bar_p);
        ok = ptx::named_bar_and(pair_bar, 64, ptx::mbar_wait_warp(bar_o, (uint32_t)(i & 1)));     // also publishes the partner's row sum
        if (!ok) break;
        ptx::tc_fence_after();
        sum += xsum[(half ^ 1) * 128 + r];
        uint32_t o0[32];
        ptx::tmem_ld32(t_s + CXT_O_COL + (uint32_t)(half * 32), o0);
        ptx::tmem_ld_wait();
        ptx::tc_fence_before();
        ptx::mbar_arrive(bar_or);                           // O (and P) may be overwritten by the next tile's scores
        const int row = i * 128 + r;
        if (row < rows) {
          const float inv = 1.0f / sum;
          uint4* o = reinterpret_cast<uint4*>(out + (size_t)(row0 + row) * d + hd * 64 + half * 32);
#pragma unroll
          for (int j = 0; j < 4; ++j)
            o[j] = make_uint4(pack_bf16x2(__uint_as_float(o0[8 * j]) * inv, __uint_as_float(o0[8 * j + 1]) * inv),
                              pack_bf16x2(__uint_as_float(o0[8 * j + 2]) * inv, __uint_as_float(o0[8 * j + 3]) * inv),
                              pack_bf16x2(__uint_as_float(o0[8 * j + 4]) * inv, __uint_as_float(o0[8 * j + 5]) * inv),
                              pack_bf16x2(__uint_as_float(o0[8 * j + 6]) * inv, __uint_as_float(o0[8 * j + 7]) * inv));
        }
      }
    }
  }
  if (!ok) {
    atomicExch(status, 5);
    const long long t0 = clock64();
    while (clock64() - t0 < 400000ll) { }      // let copies that are still in flight land before the memory is given back
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  if (warp == 8) ptx::tmem_dealloc(tmem_base, CXT_TMEM_COLS);
}

}  // namespace tsdp
