// Kernels of the speculative round that are not network forwards: chunk initialisation, the
// drafter's scheduler step (posterior mean + noise), and the fused verification tail -- posterior
// of every candidate, log acceptance ratio, decision, first-rejection scan, reflection / bonus
// commit and statistics -- in one launch.
#pragma once
#include "common.cuh"

namespace tsdp {

constexpr int TSDP_PLAN_MAXK = 32;      // = TSDP_MAX_K of the C ABI


// x_T ~ N(0, I), t = T-1 for every environment.  xt holds the round's candidate latents
// [B, Kmax+1, D]; slot 0 is the current latent x.
__global__ void init_chunk_kernel(float* __restrict__ xt, long long xs_b, int* __restrict__ t, int B, int D,
                                  int T, const uint64_t* __restrict__ seedp, int* __restrict__ round_idx, int* __restrict__ n_done,
                                  int* __restrict__ item, int* __restrict__ queue_head) {
  pdl_trigger();
  pdl_wait();
  const uint64_t seed = *seedp;
  const int b = blockIdx.x;
  const int nq = (D + 3) >> 2;
  for (int q = threadIdx.x; q < nq; q += blockDim.x) {
    float z[4];
    normal4(seed, (uint32_t)b, STREAM_INIT, 0u, (uint32_t)q, z);
#pragma unroll
    for (int j = 0; j < 4; ++j)
      if (4 * q + j < D) xt[b * xs_b + 4 * q + j] = z[j];
  }
  if (threadIdx.x == 0) {
    t[b] = T - 1;
    item[b] = b;                         // slot b starts on request b; further requests are taken from queue_head on
    if (b == 0) { *round_idx = 0; *n_done = 0; *queue_head = B; }
  }
}

// ------------------------------------------------------------------------------------------------
// Plan of a round (first kernel of the round): which candidates the base model must evaluate and which slots the
// drafter must run at each draft step, as dense lists, so that finished environments, draft slots beyond an
// environment's window K_eff = min(K, scheduler cap, t) (Sec. 3.2: drafting stops at K or at t = 0) and an unused
// bonus slot cost no network rows.
//   live_list[0 .. *live_n)       : (b << 6) | c for b ascending, c = 0 .. n_base(b) - 1,
//                                   n_base = K_eff + 1 if the bonus step can be taken (or K_eff = 0), else K_eff
//   slot_start[b], slot_start[B]  : first list entry of slot b / the total (a slot's candidates are contiguous)
//   order[0 .. dn[1])             : (b << 6) of the drafting slots, longest window first (stable in b), so that the
//                                   slots drafting at step k are the prefix order[0 .. dn[k])
//   dn[k], k = 1..K               : slots with K_eff >= k
// One block of PLAN_THREADS threads; B <= PLAN_MAX_B.
// ------------------------------------------------------------------------------------------------
constexpr int PLAN_THREADS = 1024;
constexpr int PLAN_MAX_B = 4096;
constexpr int PLAN_PER_THREAD = PLAN_MAX_B / PLAN_THREADS;

__global__ void __launch_bounds__(PLAN_THREADS)
round_plan_kernel(const int* __restrict__ t, int B, int K, const RoundParams* __restrict__ sched, int n_sched,
                  const int* __restrict__ round_idx, const EnvParams* __restrict__ envp, const int* __restrict__ item,
                  int Tsteps, int* __restrict__ live_n, int* __restrict__ live_list, int* __restrict__ slot_start,
                  int* __restrict__ order, int* __restrict__ dn, DevStats* __restrict__ stats) {
  pdl_trigger();
  pdl_wait();
  __shared__ signed char s_ke[PLAN_MAX_B];          // K_eff of each slot, -1: finished
  __shared__ int s_warp[PLAN_THREADS / 32];
  __shared__ int s_hist[TSDP_PLAN_MAXK + 2];        // slots with K_eff == k
  __shared__ int s_base[TSDP_PLAN_MAXK + 2];        // first position in `order` of the slots with K_eff == k
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int bonus = sched[min(*round_idx, n_sched - 1)].bonus;
  if (tid < TSDP_PLAN_MAXK + 2) s_hist[tid] = 0;
  __syncthreads();
  // ---- per slot: K_eff and the number of candidates the base model must see
  int nb[PLAN_PER_THREAD], mine = 0;
#pragma unroll
  for (int j = 0; j < PLAN_PER_THREAD; ++j) {
    const int b = tid * PLAN_PER_THREAD + j;
    int ke = -1, n = 0;
    if (b < B) {
      const int tb = t[b];
      if (tb >= 0) {
        ke = min(env_draft_cap(envp, item_of(item, b), tb, K, Tsteps), tb);
        n = (bonus || ke == 0) ? ke + 1 : ke;
        if (ke > 0) atomicAdd(&s_hist[ke], 1);
      }
      s_ke[b] = (signed char)ke;
    }
    nb[j] = n; mine += n;
  }
  // ---- exclusive scan of the candidate counts over the slots
  int incl = mine;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int v = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += v;
  }
  if (lane == 31) s_warp[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    int w = s_warp[lane];
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int v = __shfl_up_sync(0xffffffffu, w, o);
      if (lane >= o) w += v;
    }
    s_warp[lane] = w;                               // inclusive over warps
  }
  __syncthreads();
  int start = incl - mine + (warp > 0 ? s_warp[warp - 1] : 0);
  const int total = s_warp[PLAN_THREADS / 32 - 1];
#pragma unroll
  for (int j = 0; j < PLAN_PER_THREAD; ++j) {
    const int b = tid * PLAN_PER_THREAD + j;
    if (b < B) {
      slot_start[b] = start;
      for (int c = 0; c < nb[j]; ++c) live_list[start + c] = (b << 6) | c;
      start += nb[j];
    }
  }
  // ---- draft order: counting sort by K_eff, longest first; dn[k] = slots with K_eff >= k
  if (tid == 0) {
    slot_start[B] = total;
    *live_n = total;
    int run = 0, drafts = 0;
    for (int k = K; k >= 1; --k) { s_base[k] = run; run += s_hist[k]; dn[k] = run; drafts += run; }
    dn[0] = B;
    atomicAdd(&stats->cand_computed, (unsigned long long)total);
    atomicAdd(&stats->draft_computed, (unsigned long long)drafts);
  }
  __syncthreads();
  // warp w places the slots whose K_eff is w + 1 (K <= 32 = the number of warps), in slot order
  const int k = warp + 1;
  if (k <= K) {
    int pos = s_base[k];
    for (int b0 = 0; b0 < B; b0 += 32) {
      const int b = b0 + lane;
      const bool hit = b < B && s_ke[b] == k;
      const unsigned m = __ballot_sync(0xffffffffu, hit);
      if (hit) order[pos + __popc(m & ((1u << lane) - 1u))] = b << 6;
      pos += __popc(m);
    }
  }
}

// Draft step k (Eq. (3) of Sec. 3.2): tau = t - k + 1, mu^_k = posterior mean of (x~_{k-1}, eps^),
// x~_k = mu^_k + sigma_tau xi_tau.  Slots beyond K_eff = min(K, t) copy the previous latent so that
// every buffer stays finite.  eps^ of slot b is the D values at eps_d + b * es_b.
__global__ void draft_step_kernel(DdpmTables S, float* __restrict__ xt, long long xs_b, float* __restrict__ muhat,
                                  long long ms_b, const float* __restrict__ eps_d, long long es_b, const int* __restrict__ t,
                                  int k, int D, const uint64_t* __restrict__ seedp, const EnvParams* __restrict__ envp,
                                  int K, int Tsteps, const int* __restrict__ item) {
  pdl_trigger();
  pdl_wait();
  const uint64_t seed = *seedp;
  const int b = blockIdx.x;
  const int tb = t[b];
  const int tau = tb - k + 1;
  const int env = item_of(item, b);      // the request this slot serves: index of its noise streams and parameters
  const bool valid = (tb >= 0) && (tau >= 1) && (k <= env_draft_cap(envp, env, tb, K, Tsteps));
  const float* xp = xt + b * xs_b + (long long)(k - 1) * D;
  float* xn = xt + b * xs_b + (long long)k * D;
  float* mh = muhat + b * ms_b + (long long)(k - 1) * D;
  const float* e = eps_d + b * es_b;
  const int nq = (D + 3) >> 2;
  for (int q = threadIdx.x; q < nq; q += blockDim.x) {
    float z[4] = {0.f, 0.f, 0.f, 0.f};
    if (valid) normal4(seed, (uint32_t)env, STREAM_XI, (uint32_t)tau, (uint32_t)q, z);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int i = 4 * q + j;
      if (i < D) {
        const float x = xp[i];
        if (valid) {
          const float m = posterior_mean(S, x, e[i], tau);
          mh[i] = m;
          xn[i] = ddpm_sample(m, S.sigma[tau], z[j]);
        } else {
          mh[i] = x;
          xn[i] = x;
        }
      }
    }
  }
}

// Four consecutive latent values starting at element 4q: one 16-byte load when D is a multiple of 4 (every row of
// the round's buffers then starts on a 16-byte boundary), element by element with a bounds check otherwise.
__device__ __forceinline__ void load_quad(const float* __restrict__ p, int q, int D, bool vec, float v[4]) {
  if (vec) {
    const float4 t = *reinterpret_cast<const float4*>(p + 4 * q);
    v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
  } else {
#pragma unroll
    for (int j = 0; j < 4; ++j) v[j] = 4 * q + j < D ? p[4 * q + j] : 0.f;
  }
}
__device__ __forceinline__ void store_quad(float* __restrict__ p, int q, int D, bool vec, const float v[4]) {
  if (vec) *reinterpret_cast<float4*>(p + 4 * q) = make_float4(v[0], v[1], v[2], v[3]);
  else {
#pragma unroll
    for (int j = 0; j < 4; ++j)
      if (4 * q + j < D) p[4 * q + j] = v[j];
  }
}

// Fused verification tail, one block per environment, one warp per drafted step.
//   warp k-1 (k = 1..K_eff): mu_k = posterior mean of (x~_{k-1}, eps_{k-1}) at tau = t-k+1;
//       d = (mu^_k - mu_k) / (s sigma_tau);  log alpha = -1/2 |d|^2 - <d, xi_tau>   (Sec. 3.2)
//       accept iff log alpha >= log U_tau (mode 0) or min(0, log alpha) >= log lambda (mode 1).
//   thread 0: j* = first rejected step (Sec. 3.1 Eq. (3)), statistics.
//   all threads: commit -- reflection x = mu + (I - 2 e e^T)(x~ - mu^) at j* (Sec. 3.1), or the bonus
//       base step, or the last draft -- into slot 0; t -= steps; finished chunks go to `actions`.
// `item` maps the slot to the request it serves (null: the slot index), `queue_head` / `n_items` feed
// finished slots with waiting requests (null: no refill).  item_counts (may be null) holds four
// counters per request -- drafts proposed, drafts accepted, rounds, reverse steps taken -- the inputs of
// the intermediate reward of Sec. 3.3.  dbg_* may be null.
__global__ void accept_kernel(DdpmTables S, float* __restrict__ xt, long long xs_b,
                              const float* __restrict__ muhat, long long ms_b,
                              const float* __restrict__ eps, long long es_b, int* __restrict__ t, int K, int D,
                              const uint64_t* __restrict__ seedp, const RoundParams* __restrict__ sched, int n_sched,
                              const int* __restrict__ round_idx, float* __restrict__ actions,
                              int* __restrict__ n_done, DevStats* __restrict__ stats, float draft_nfe,
                              float* __restrict__ dbg_logalpha, int* __restrict__ dbg_jstar,
                              const EnvParams* __restrict__ envp, int* __restrict__ item, int* __restrict__ queue_head,
                              const int* __restrict__ n_items, int* __restrict__ item_counts) {
  pdl_trigger();
  pdl_wait();
  __shared__ float s_la[32], s_s1[32], s_s2[32];
  __shared__ int s_acc[32];
  __shared__ int s_j;
  const uint64_t seed = *seedp;
  const int b = blockIdx.x;
  const int tb = t[b];
  if (tb < 0) {
    if (dbg_jstar && threadIdx.x == 0) dbg_jstar[b] = -1;
    return;
  }
  const int r = min(*round_idx, n_sched - 1);
  RoundParams rp = sched[r];
  const int env = item_of(item, b);      // the request this slot serves
  if (envp) { rp.sigma_scale = envp[env].sigma_scale; rp.log_lambda = envp[env].log_lambda; }   // the scheduler's choice
  const int K_eff = min(env_draft_cap(envp, env, tb, K, S.T), tb);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nq = (D + 3) >> 2;
  const float* xb = xt + b * xs_b;
  const float* mb = muhat + b * ms_b;
  const float* eb = eps + b * es_b;
  // 16-byte loads when every row of the three buffers is 16-byte aligned
  const bool vec = (D & 3) == 0 && (xs_b & 3) == 0 && (ms_b & 3) == 0 && (es_b & 3) == 0 &&
                   ((reinterpret_cast<uintptr_t>(xt) | reinterpret_cast<uintptr_t>(muhat) | reinterpret_cast<uintptr_t>(eps) |
                     reinterpret_cast<uintptr_t>(actions)) & 15) == 0;

  for (int k = warp + 1; k <= K_eff; k += (blockDim.x >> 5)) {
    const int tau = tb - k + 1;
    const float inv = 1.0f / (rp.sigma_scale * S.sigma[tau]);
    float s1 = 0.f, s2 = 0.f, d2 = 0.f;
    for (int q = lane; q < nq; q += 32) {
      float z[4], xv[4], ev[4], mv[4];
      normal4(seed, (uint32_t)env, STREAM_XI, (uint32_t)tau, (uint32_t)q, z);
      load_quad(xb + (long long)(k - 1) * D, q, D, vec, xv);
      load_quad(eb + (long long)(k - 1) * D, q, D, vec, ev);
      load_quad(mb + (long long)(k - 1) * D, q, D, vec, mv);
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int i = 4 * q + j;
        if (i < D) {
          const float mu = posterior_mean(S, xv[j], ev[j], tau);
          const float delta = mv[j] - mu;
          const float d = delta * inv;
          s1 += d * d; s2 += d * z[j]; d2 += delta * delta;
        }
      }
    }
    s1 = warp_sum(s1); s2 = warp_sum(s2); d2 = warp_sum(d2);
    if (lane == 0) {
      const float la = -0.5f * s1 - s2;
      bool acc;
      if (d2 < 1e-30f) acc = true;
      else if (rp.mode == 0) acc = la >= logf(uniform1(seed, (uint32_t)env, (uint32_t)tau));
      else acc = fminf(0.f, la) >= rp.log_lambda;
      s_la[k - 1] = la; s_s1[k - 1] = s1; s_s2[k - 1] = s2; s_acc[k - 1] = acc ? 1 : 0;
      if (dbg_logalpha) dbg_logalpha[b * K + (k - 1)] = la;
    }
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    int j = K_eff + 1;
    for (int k = 1; k <= K_eff; ++k)
      if (!s_acc[k - 1]) { j = k; break; }
    s_j = j;
    if (dbg_jstar) dbg_jstar[b] = j;
    if (dbg_logalpha)
      for (int k = K_eff + 1; k <= K; ++k) dbg_logalpha[b * K + (k - 1)] = 0.f;
  }
  __syncthreads();
  const int j = s_j;
  const bool rejected = j <= K_eff;
  const bool bonus = !rejected && (rp.bonus || K_eff == 0);
  const int adv = rejected ? j : (bonus ? K_eff + 1 : K_eff);
  const int t_new = tb - adv;
  float* xo = xt + b * xs_b;   // slot 0
  if (rejected) {
    const int tau = tb - j + 1;
    const float sig = S.sigma[tau];
    // e <e, xi> = Delta <Delta, xi> / |Delta|^2 = Delta * S2 / (S1 * s * sigma)
    const float coef = 2.0f * s_s2[j - 1] / (s_s1[j - 1] * rp.sigma_scale * sig);
    for (int q = threadIdx.x; q < nq; q += blockDim.x) {
      float z[4], xv[4], ev[4], mv[4], ov[4] = {0.f, 0.f, 0.f, 0.f};
      normal4(seed, (uint32_t)env, STREAM_XI, (uint32_t)tau, (uint32_t)q, z);
      load_quad(xb + (long long)(j - 1) * D, q, D, vec, xv);
      load_quad(eb + (long long)(j - 1) * D, q, D, vec, ev);
      load_quad(mb + (long long)(j - 1) * D, q, D, vec, mv);
#pragma unroll
      for (int jj = 0; jj < 4; ++jj) {
        const float mu = posterior_mean(S, xv[jj], ev[jj], tau);
        const float delta = mv[jj] - mu;
        ov[jj] = mu + sig * (z[jj] - coef * delta);
      }
      store_quad(xo, q, D, vec, ov);
      if (t_new < 0) store_quad(actions + (long long)env * D, q, D, vec, ov);
    }
  } else if (bonus) {
    const int tau = tb - K_eff;
    const float sig = S.sigma[tau];
    for (int q = threadIdx.x; q < nq; q += blockDim.x) {
      float z[4] = {0.f, 0.f, 0.f, 0.f}, xv[4], ev[4], ov[4];
      if (tau > 0) normal4(seed, (uint32_t)env, STREAM_XI, (uint32_t)tau, (uint32_t)q, z);
      load_quad(xb + (long long)K_eff * D, q, D, vec, xv);
      load_quad(eb + (long long)K_eff * D, q, D, vec, ev);
#pragma unroll
      for (int jj = 0; jj < 4; ++jj) ov[jj] = ddpm_sample(posterior_mean(S, xv[jj], ev[jj], tau), sig, z[jj]);
      store_quad(xo, q, D, vec, ov);
      if (t_new < 0) store_quad(actions + (long long)env * D, q, D, vec, ov);
    }
  } else {
    for (int i = threadIdx.x; i < D; i += blockDim.x) {
      const float v = xb[(long long)K_eff * D + i];
      xo[i] = v;
      if (t_new < 0) actions[(long long)env * D + i] = v;
    }
  }
  if (threadIdx.x < 32) {      // statistics: the lanes of warp 0 issue the independent atomics side by side
    const int n_acc = min(j - 1, K_eff);
    const int n_tested = min(j, K_eff);
    const unsigned long long vals[9] = {1ull, (unsigned long long)((rp.bonus || K_eff == 0) ? K_eff + 1 : K_eff),
                                        (unsigned long long)K_eff, (unsigned long long)n_tested, (unsigned long long)n_acc,
                                        rejected ? 1ull : 0ull, bonus ? 1ull : 0ull, (unsigned long long)adv, K_eff > 0 ? 1ull : 0ull};
    unsigned long long* ctr[9] = {&stats->env_rounds, &stats->base_evals, &stats->draft_evals, &stats->drafts_tested,
                                  &stats->drafts_accepted, &stats->rejections, &stats->bonus_steps, &stats->steps_advanced,
                                  &stats->draft_rounds};
    if (threadIdx.x < 9 && vals[threadIdx.x] != 0ull) atomicAdd(ctr[threadIdx.x], vals[threadIdx.x]);
    for (int k = 1 + (int)threadIdx.x; k <= K_eff; k += 32) {
      const int tau = tb - k + 1;
      atomicAdd(&stats->hist_drafted[tau], 1ull);
      if (k <= n_tested) atomicAdd(&stats->hist_tested[tau], 1ull);
      if (k <= n_acc) atomicAdd(&stats->hist_accepted[tau], 1ull);
    }
  }
  if (threadIdx.x == 0) {
    t[b] = t_new;
    const int n_acc = min(j - 1, K_eff);
    if (item_counts) {                     // a request occupies one slot at a time: no atomics needed
      int* ic = item_counts + 4 * (long long)env;
      ic[0] += K_eff; ic[1] += n_acc; ic[2] += 1; ic[3] += adv;
    }
    if (t_new < 0) {
      atomicAdd(&stats->chunks_done, 1ull);
      atomicAdd(n_done, 1);
    }
  }
  // Continuous batching: a slot whose request has finished takes the next waiting request, if any --
  // fresh x_T ~ N(0, I) from that request's own noise stream, t = T - 1.
  if (t_new < 0 && queue_head != nullptr) {
    __shared__ int s_next;
    __syncthreads();                       // the committed latent above has been written and read
    if (threadIdx.x == 0) s_next = atomicAdd(queue_head, 1);
    __syncthreads();
    const int next = s_next;
    if (next < *n_items) {
      for (int q = threadIdx.x; q < nq; q += blockDim.x) {
        float z[4];
        normal4(seed, (uint32_t)next, STREAM_INIT, 0u, (uint32_t)q, z);
#pragma unroll
        for (int jj = 0; jj < 4; ++jj)
          if (4 * q + jj < D) xo[4 * q + jj] = z[jj];
      }
      if (threadIdx.x == 0) { item[b] = next; t[b] = S.T - 1; }
    }
  }
}

// Intermediate ("process") reward of the scheduler's training signal, Sec. 3.3 "Reward function":
//   r = (n_accept / n_draft + n_accept / n_diffusion) * lambda,  lambda = (R_final / 4) / ceil(T_max / dt),
// per request, from the counters the acceptance kernel keeps.  A ratio with a zero denominator counts 0.
__global__ void process_reward_kernel(const int* __restrict__ item_counts, int n, float R_final, int T_max, int dt,
                                      float* __restrict__ reward) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  const int n_draft = item_counts[4 * i], n_acc = item_counts[4 * i + 1], n_diff = item_counts[4 * i + 3];
  const int n_expected = (T_max + dt - 1) / dt;
  const float lam = (0.25f * R_final) / (float)n_expected;
  const float a = n_draft > 0 ? (float)n_acc / (float)n_draft : 0.f;
  const float e = n_diff > 0 ? (float)n_acc / (float)n_diff : 0.f;
  reward[i] = (a + e) * lam;
}

// End of a round: advance the schedule index and publish the number of finished chunks where the
// host can read it.
__global__ void round_end_kernel(int* __restrict__ round_idx, const int* __restrict__ n_done,
                                 volatile int* __restrict__ host_done) {
  pdl_trigger();
  pdl_wait();
  *round_idx += 1;
  *host_done = *n_done;
}

}  // namespace tsdp
