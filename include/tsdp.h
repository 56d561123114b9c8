/* tsdp.h -- C ABI of the B200 (sm_100a) implementation of the TS-DP speculative denoising loop for
 * Diffusion Policy (arXiv 2512.15773).
 *
 * One context samples action chunks for up to max_B independent environments.  One chunk is T DDPM
 * reverse steps, taken in speculative rounds (Sec. 3.2 of the paper):
 *   1. the drafter rolls out K reverse steps with the shared DDPM scheduler         (Eq. (3));
 *   2. the base denoiser is evaluated on all K+1 candidate latents of every environment in one
 *      batched forward                                         ("Verification of Speculative Drafts");
 *   3. per drafted step the Gaussian log acceptance ratio  log a = -1/2 |d|^2 - <d, xi>,
 *      d = (mu^ - mu) / (s sigma)  is tested, the accepted prefix is committed, and the first rejected
 *      step is replaced by its reflection-maximal coupling             (Sec. 3.1, Eqs. (1)-(3) and the
 *      reflection equations).
 *
 * Conventions.  All pointers named d_* are DEVICE pointers, h_* are HOST pointers.  Arrays are dense,
 * row-major, fp32 unless stated.  Timestep t in {T-1..0}: a network called with t receives the latent
 * "at t"; the transition at t produces the latent at t-1; the latent at -1 is the clean action chunk.
 * Kernels of a round are chained with programmatic dependent launch (each may start its prologue while
 * its predecessor drains); setting the environment variable TSDP_NO_PDL before tsdp_init turns that off.
 * In bf16 the decoder transformer (TSDP_ARCH_XFMR) runs the cross-attention sub-block of every block folded
 * into its memory tokens (the query and output projections are applied once to the time / observation tokens
 * instead of to every token row) when H <= 16, (1 + obs_tokens) * heads <= 32, heads is even and d is 128, 256
 * or 512; TSDP_NO_FOLD, set before tsdp_load_weights, keeps the separate kernels.  Same function either way.
 * TSDP_NO_ASYNC_BCAST (read by tsdp_init, like TSDP_NO_PDL) makes the cluster kernel hand its stages over with plain distributed-
 * shared-memory stores and a cluster barrier instead of st.async stores counted by mbarriers.
 * TSDP_GEMM_PAIR = 0 | 1 | 2 (read by tsdp_init; default 1) selects the two-CTA form of the tensor-core GEMM
 * (tcgen05 cta_group::2, 256 x 256 tiles on clusters of two CTAs): never / for long reductions with enough tiles /
 * wherever the output width allows -- a tuning aid; results do not depend on it.
 * TSDP_GEMM_BN = 32 | 64 | 128 | 256 (read by tsdp_init) forces that tile width on every tensor-core GEMM whose
 * output width it divides -- a tuning aid; results do not depend on the tile width.
 * Further switches, all read by tsdp_init unless stated, none of which changes what is computed (they select between
 * kernels that are tested against the same reference): TSDP_NO_COMPACT runs every round on the dense candidate
 * layout instead of the list of live candidates; TSDP_NO_FUSED_ATTN (read at every forward) keeps the 16-token
 * self-attention as a kernel of its own instead of the QKV projection's epilogue; TSDP_NO_TC_ATTN keeps the context
 * cross-attention of TSDP_ARCH_DIT on the mma.sync kernel, TSDP_TC_ATTN=2 puts it on the tcgen05 kernel for every
 * group size (default: groups of at least 256 query rows, 64-wide heads, obs_tokens a multiple of 32 and <= 256);
 * TSDP_NO_KSPLIT keeps the convolution GEMMs of TSDP_ARCH_UNET from splitting their reduction over idle SMs at small
 * batch (the split changes the order of the fp32 sums, so the last bits of a result depend on it; for a given
 * batch shape the result is the same on every run);
 * TSDP_NO_AUX_STREAM keeps the 1x1 residual convolutions of TSDP_ARCH_UNET on the caller's stream instead of a second
 * stream of the context beside the block's two kernel-5 convolutions (inside the round's CUDA graph: a parallel branch);
 * TSDP_VERBOSE prints the kernels' occupancy figures once per tsdp_load_weights.
 * Every function returns a tsdp_status; nothing throws or aborts.  A context is not re-entrant: one
 * call at a time.  There is no CPU fallback: without a CUDA device tsdp_init fails with TSDP_ERR_CUDA.
 */
#ifndef TSDP_H
#define TSDP_H
#include <stddef.h>
#include <stdint.h>
#ifdef __cplusplus
extern "C" {
#endif

typedef struct tsdp_ctx tsdp_ctx; /* opaque; owned by the library */

typedef enum {
  TSDP_OK = 0,
  TSDP_ERR_ARG = 1,         /* null pointer, size out of range, unsupported shape          */
  TSDP_ERR_STATE = 2,       /* weights not loaded yet                                      */
  TSDP_ERR_WEIGHTS = 3,     /* blob size does not match the configured architecture        */
  TSDP_ERR_CUDA = 4,        /* a CUDA runtime / driver call failed (see tsdp_last_error)   */
  TSDP_ERR_TIMEOUT = 5,     /* a bounded wait inside a kernel expired                      */
  TSDP_ERR_NAN = 6,         /* non-finite value in a weight blob                           */
  TSDP_ERR_UNSUPPORTED = 7, /* architecture not built                                      */
  TSDP_ERR_TOO_LARGE = 8,   /* size beyond the capacity of tsdp_verify_commit_static       */
  TSDP_ERR_OVERRUN = 9      /* tsdp_debug_check_guards found a buffer overrun              */
} tsdp_status;

enum { TSDP_ARCH_GAUSS = 0, TSDP_ARCH_MLP = 1, TSDP_ARCH_XFMR = 2, TSDP_ARCH_DIT = 3, TSDP_ARCH_UNET = 4,
       /* Only as the DRAFT network: no drafter at all.  The drafts of a round reuse the base model's output at
        * the round's starting latent for every step ("frozen target draft", the drafter-free scheme of the prior
        * work cited in Sec. 2.2): eps^_k = eps_base(x, t) for k = 1..K.  A round then costs one base forward on
        * the B current latents plus the batched verification; the first draft is the base model's own step and
        * is always accepted.  Takes no weights: tsdp_load_weights(TSDP_DRAFT) is not called. */
       TSDP_ARCH_FROZEN = 5 };
enum { TSDP_BASE = 0, TSDP_DRAFT = 1, TSDP_SCHED = 2 };
enum { TSDP_MAX_T = 1024, TSDP_MAX_K = 32, TSDP_LATENCY_RING = 256 };

/* One denoiser eps = M(x, t; obs).
 *   GAUSS: closed-form optimal denoiser of iid N(m0, s0^2) data (the 1-D Gaussian toy); no sizes.
 *   MLP  : input [latent | sinusoidal(t, temb) | obs], `layers` hidden SiLU layers of width `d`.
 *   XFMR : pre-LN decoder, `layers` blocks [causal self-attn, cross-attn to (time token | obs tokens),
 *          GELU MLP 4d], model width `d` (multiple of 128), `heads` heads (d/heads multiple of 32).
 *   DIT  : adaptive-LayerNorm transformer: the timestep enters each of the `layers` blocks as shift /
 *          scale / gate vectors, the obs_tokens (<= 256) observation/context tokens through
 *          cross-attention, self-attention over the H action tokens is bidirectional;
 *          h += g1 * SelfAttn(LN0(h)(1+k1)+s1) Wo;  h += CrossAttn(LN(h), ctx) Wo2;  h += g2 * MLP(LN0(h)(1+k2)+s2).
 *   UNET : 1-D temporal conv UNet over the H action positions: `layers` levels with d, 2d, 4d.. channels, two
 *          FiLM residual blocks per level (conv k5 -> GroupNorm(`heads` groups) -> Mish, FiLM scale/bias from
 *          Mish([time vector (temb wide) | flattened obs])), 2:1 mean pooling down, 2x repetition up, skip
 *          concatenation, two middle blocks, conv + pointwise head.  H a multiple of 2^(layers-1).
 * The paper fixes only the block counts (8 for the base policy, 1 for the drafter; Sec. 4). */
typedef struct {
  int arch, layers, d, heads, temb;
} tsdp_net_t;

typedef struct {
  tsdp_net_t base, draft;
  int H, A;                /* action horizon and action dimension; latent size D = H*A        */
  int obs_tokens, obs_dim; /* observation: obs_tokens x obs_dim features per environment       */
  int T;                   /* DDPM steps (paper: 100), <= TSDP_MAX_T                          */
  float beta0, beta1;      /* linear beta schedule                                            */
  float clip;              /* clamp x0_hat to +-clip when > 0                                  */
  int max_B, max_K;        /* capacity: environments per call, draft steps per round          */
  int precision;           /* 0: fp32 check mode (CUDA cores); 1: bf16 tensor-core mode       */
  int device;              /* CUDA device ordinal                                              */
  float draft_nfe;         /* NFE cost of one drafter call; 0 => draft.layers/base.layers
                              (the paper's 1/8 rule, Sec. 4 "Evaluation Metrics")               */
  int use_graph;           /* 1: replay each round from a captured CUDA graph                  */
  int drafter;             /* how the K draft steps run.  0: chosen from the batch size; 1: layer
                              by layer (batched tensor-core kernels, one drafter forward per step);
                              2: one persistent thread-block-cluster kernel per round with the
                              drafter's weights sliced over the 8 CTAs of the cluster: resident
                              in shared memory when a 1/8 slice fits beside the activations, read
                              through the L2 otherwise (transformer drafter, precision 1, d = 128
                              or 256, <= 4 blocks, H <= 16, obs_tokens <= 3; otherwise tsdp_init
                              returns UNSUPPORTED)                                               */
  int verifier;            /* how the base model's verification forward runs.  0: chosen from the
                              number of candidates; 1: batched tensor-core kernels, layer by layer;
                              2: the cluster kernel above, one cluster per candidate, in one launch
                              (same shape limits, <= 8 blocks; meant for batch 1, where the
                              layer-by-layer forward is bound by the latency of ~90 small launches) */
} tsdp_config_t;

/* Speculative parameters of a round -- the scheduler's action space (Sec. 3.3).
 *   mode 0: accept iff U <= min(1, alpha)  (lossless likelihood-ratio test, Sec. 3.1 Eq. (2));
 *   mode 1: accept iff min(1, alpha) >= lambda, lambda in (0,1]  (the threshold rule of Sec. 3.2).
 *   sigma_scale s >= 1 widens only the test statistic, d = (mu^ - mu)/(s sigma).
 *   bonus 1: when no draft is rejected the base model's evaluation of the last draft is used for one
 *            more reverse step (K+1 candidates verified); 0: only the K drafted latents count. */
typedef struct {
  int mode;
  float lambda;
  float sigma_scale;
  int bonus;
} tsdp_accept_t;

typedef struct {
  uint64_t chunks;          /* environment-chunks completed                                   */
  uint64_t rounds;          /* batched rounds launched                                        */
  uint64_t env_rounds;      /* rounds summed over environments (= batched base forwards each saw) */
  uint64_t base_evals;      /* candidate latents the base model evaluated (useful ones)       */
  uint64_t draft_evals;     /* drafter calls (= drafts proposed)                               */
  uint64_t drafts_tested, drafts_accepted, rejections, bonus_steps, steps_advanced;
  uint64_t draft_rounds;    /* rounds summed over environments in which at least one step was drafted */
  double nfe;               /* env_rounds + draft_nfe * draft_evals (+ draft_rounds with TSDP_ARCH_FROZEN drafts:
                               the base forward that supplies them)                            */
  uint64_t hist_drafted[TSDP_MAX_T], hist_tested[TSDP_MAX_T], hist_accepted[TSDP_MAX_T];
                            /* per timestep of the drafted transition                          */
  /* Device time (CUDA events on the caller's stream, copies included) of the last calls of
   * tsdp_sample_chunk / tsdp_sample_chunk_host / tsdp_serve since the last reset, kept in a ring of
   * TSDP_LATENCY_RING entries: nearest-rank median and 99th percentile in milliseconds, and how
   * many calls they are taken over (0: no call yet, percentiles are 0).  With one environment per
   * call this is the per-chunk latency the paper's Table 5 reports. */
  double call_ms_p50, call_ms_p99;
  uint64_t call_ms_samples;
  /* Candidate latents the verification forwards covered.  cand_dense: what the dense layout B x (K+1) per round
   * amounts to; cand_computed: what was really evaluated -- each round first lists the candidates that are still
   * needed (unfinished environments, draft slots up to K_eff, the bonus slot) and the layer-by-layer forwards run
   * on that list only (TSDP_NO_COMPACT, read by tsdp_init, or more than 4096 environments per call: dense).
   * Rounds verified by the cluster kernel count in cand_dense only. */
  uint64_t cand_dense, cand_computed;
} tsdp_stats_t;

/* Create a context on cfg->device: allocates every workspace for (max_B, max_K).  *out is set only on
 * success.  Errors: ARG (bad sizes), UNSUPPORTED (arch), CUDA. */
int tsdp_init(const tsdp_config_t* cfg, tsdp_ctx** out);
void tsdp_destroy(tsdp_ctx* ctx);
const char* tsdp_strerror(int status);
/* Text of the last CUDA failure seen by this context ("" if none); valid until the next call. */
const char* tsdp_last_error(const tsdp_ctx* ctx);

/* Number of fp32 values tsdp_load_weights expects for net `which` (0 on a bad argument). */
size_t tsdp_weights_count(const tsdp_config_t* cfg, int which);

/* Load a denoiser from a HOST blob of n fp32 values, copied during the call (caller keeps ownership).
 * Linear layers y = x W + b are stored W [in, out] row-major then b [out].  Order:
 *   GAUSS: m0, s0.
 *   MLP  : (W, b) for each hidden layer, then the head.  in = H*A + temb + obs_tokens*obs_dim.
 *   XFMR : W_in [A,d], b_in, pos [H,d], W_obs [obs_dim,d], b_obs, cpos [1+obs_tokens,d];
 *          per block: ln1_g, ln1_b, Wqkv [d,3d], bqkv, Wo, bo, ln2_g, ln2_b, Wq2, bq2, Wkv2 [d,2d], bkv2,
 *                     Wo2, bo2, ln3_g, ln3_b, W1 [d,4d], b1, W2 [4d,d], b2;
 *          lnf_g, lnf_b, W_out [d,A], b_out.
 *   DIT  : W_in [A,d], b_in, pos [H,d], W_ctx [obs_dim,d], b_ctx, cpos [obs_tokens,d], Wt1 [d,d], bt1, Wt2 [d,d], bt2;
 *          per block: Wmod [d,6d], bmod (shift1, scale1, gate1, shift2, scale2, gate2), Wqkv, bqkv, Wo, bo,
 *                     lnc_g, lnc_b, Wq2, bq2, Wkv2 [d,2d], bkv2, Wo2, bo2, W1, b1, W2, b2;
 *          Wmodf [d,2d], bmodf (shift, scale of the final layer), W_out [d,A], b_out.
 *          The time path (Wt*, Wmod*) is kept in fp32 and tabulated for every timestep during the load.
 *   UNET : W_in [A,d], b_in, Wt1 [temb,4temb], bt1, Wt2 [4temb,temb], bt2; per residual block (C_in, C_out) in
 *          execution order: W1 [5,C_in,C_out] (tap, in, out), b1, g1, be1, Wf [temb+obs_tokens*obs_dim, 2C_out], bf,
 *          W2 [5,C_out,C_out], b2, g2, be2, and if C_in != C_out: Wr [C_in,C_out], br;
 *          Wh [5,d,d], bh, gh, beh, W_out [d,A], b_out.  The time path and the FiLM layers stay fp32 (tabulated).
 *   SCHED (which = TSDP_SCHED, the scheduler network of Sec. 3.3, always fp32): W_o [obs_tokens*obs_dim, 64],
 *          b_o, W_a [H*A, 64], b_a, W_p [1, 16], b_p, W_1 [144, 64], b_1, W_2 [64, 5], b_2.
 * In precision 1 the large matrices are rounded to bf16.  Errors: WEIGHTS (n mismatch), NAN, CUDA. */
int tsdp_load_weights(tsdp_ctx* ctx, int which, const float* h_blob, size_t n);

/* Per-round overrides for the following chunks: round r uses K_per_round[min(r, n-1)] and
 * per_round[min(r, n-1)]; n = 0 clears the schedule (every round then uses the arguments of
 * tsdp_sample_chunk).  Stands in for the RL scheduler's output (Sec. 3.3).  HOST arrays, copied. */
int tsdp_set_schedule(tsdp_ctx* ctx, const int* h_K_per_round, const tsdp_accept_t* h_per_round, int n);

/* Scheduler network (Sec. 3.3 "Temporal-Complexity-Aware Speculative Decoding Scheduler").  Inputs per
 * environment: its observation, the action chunk sampled for it last time (zeros before the first chunk)
 * and its task progress in [0, 1]; three stream encoders, an aggregating MLP, five outputs:
 *   sigma_scale = 1 + 2 sigmoid(y0),  lambda = sigmoid(y1),  K_stage = 1 + rint((max_K - 1) sigmoid(y_{2+stage}))
 * for the stages early (t >= 4T/5), middle, late (t < T/5).  Sizes and squashing are this library's own;
 * the paper names the streams, the encoders, the MLP and the outputs only.
 * While enabled, tsdp_sample_chunk evaluates the network once per chunk (on a side stream, beside the
 * chunk set-up) and every environment then uses its own sigma_scale, lambda and per-stage draft cap:
 * K_eff = min(K of the round, K_stage, t).  mode and bonus still come from the `accept` argument.
 * tsdp_set_scheduler: STATE if no TSDP_SCHED weights are loaded.  tsdp_set_progress copies B HOST floats. */
int tsdp_set_scheduler(tsdp_ctx* ctx, int enable);
int tsdp_set_progress(tsdp_ctx* ctx, const float* h_progress, int B);
/* Evaluate the scheduler network alone (test interface; synchronous).  d_obs [B, obs_tokens, obs_dim] and
 * d_prev_actions [B, H*A] DEVICE, h_progress [B] HOST; h_params [B, 8] HOST receives
 * sigma_scale, lambda, K_early, K_mid, K_late, then the three draft counts before rounding. */
int tsdp_sched_eval(tsdp_ctx* ctx, const float* d_obs, const float* d_prev_actions, const float* h_progress, int B,
                    float* h_params, void* cuda_stream);

/* Sample one action chunk for each of B environments (the whole hot path: init, rounds until every
 * environment reaches t = -1).  d_obs [B, obs_tokens, obs_dim] and d_actions [B, H, A] are DEVICE
 * buffers owned by the caller; work is enqueued on `cuda_stream` (a cudaStream_t, may be 0) and the
 * call returns after the chunk has finished (it reads a completion flag between rounds).  The same
 * (weights, obs, seed, K, accept, schedule) always gives the same chunk.
 * Errors: ARG, STATE, CUDA, TIMEOUT. */
int tsdp_sample_chunk(tsdp_ctx* ctx, const float* d_obs, int B, int K, const tsdp_accept_t* accept,
                      uint64_t seed, float* d_actions, void* cuda_stream);

/* Continuous batching: N requests (one action chunk each; d_obs [N, obs_tokens, obs_dim], d_actions [N, H, A],
 * DEVICE) are worked through `slots` <= max_B batch slots.  A slot whose request reaches t = -1 takes the
 * next waiting request inside the acceptance kernel (fresh x_T, t = T-1), so no slot idles while work
 * remains.  Request i draws the noise streams of environment i: its chunk equals the one
 * tsdp_sample_chunk returns for environment i of a batch of N with the same seed -- bit for bit when both calls run
 * the same kernels with sums in the same order (the networks are evaluated row by row); where the kernel choice or a
 * split reduction depends on the number of slots (cluster kernels at small batches, TSDP_ARCH_UNET convolutions at
 * small batches) the two agree to rounding only.  Per-request buffers grow
 * on demand (the only call besides tsdp_init / tsdp_load_weights that may allocate).  With a per-round
 * schedule the round index counts batched rounds of the whole call.  Errors as tsdp_sample_chunk. */
int tsdp_serve(tsdp_ctx* ctx, const float* d_obs, int N, int slots, int K, const tsdp_accept_t* accept,
               uint64_t seed, float* d_actions, void* cuda_stream);

/* The same with HOST buffers: copies h_obs to the device, samples, copies the chunk back. */
int tsdp_sample_chunk_host(tsdp_ctx* ctx, const float* h_obs, int B, int K, const tsdp_accept_t* accept,
                           uint64_t seed, float* h_actions);

/* One speculative round from a given state, with every intermediate exposed (test interface).
 *   d_x [B, D] in/out: current latents;  h_t [B] in/out: their timesteps (HOST).
 * Optional outputs (null to skip): d_xtilde [B, K+1, D] candidates (slot 0 = input latent),
 * d_muhat [B, K, D] drafter means, d_eps [B, K+1, D] base outputs, d_logalpha [B, K] (entries of draft
 * slots beyond an environment's window K_eff = min(K, t) are unspecified in the first three, 0 in the last),
 * h_jstar [B] (HOST; first rejected step, K_eff+1 if none, -1 if the environment was finished).
 * Synchronous. */
int tsdp_round(tsdp_ctx* ctx, const float* d_obs, int B, int K, const tsdp_accept_t* accept, uint64_t seed,
               float* d_x, int* h_t, float* d_xtilde, float* d_muhat, float* d_eps, float* d_logalpha,
               int* h_jstar, void* cuda_stream);

/* eps = M_which(x_n, tau_n; obs_n) for n < N <= max_B (test interface).  d_x, d_eps [N, D];
 * h_tau [N] HOST; d_obs [N, obs_tokens, obs_dim].  Synchronous. */
int tsdp_denoise(tsdp_ctx* ctx, int which, const float* d_x, const int* h_tau, const float* d_obs, int N,
                 float* d_eps, void* cuda_stream);

/* C[M,N] = A[M,K] W[N,K]^T + bias through the context's GEMM (tcgen05 in precision 1, where d_A, d_W
 * are bf16 and K % 64 == 0, N % 32 == 0; CUDA cores in precision 0, where they are fp32).
 * epi: 0 store (bf16 / fp32 by precision), 1 GELU then store, 2 d_out fp32 += result, 3 store fp32,
 * 4 (precision 1, N = 3K, K % 64 = 0, M % 16 = 0) the fused QKV projection + causal self-attention over chunks of
 *   16 rows with 64-wide heads: W rows (output features) ordered head by head, [Q_h | K_h | V_h] of 64 each; d_out is
 *   the attention output, bf16 [M, K].
 * Test interface; synchronous. */
int tsdp_gemm(tsdp_ctx* ctx, const void* d_A, const void* d_W, const float* d_bias, int M, int N, int K,
              int epi, void* d_out, void* cuda_stream);

/* Memory check without a memory checker (test interface).  Every device buffer a context owns -- round state, network
 * workspaces, weights, tables, plans -- is followed by 256 guard bytes holding a pattern.  This call waits for the
 * device and verifies all of them: TSDP_OK, or TSDP_ERR_OVERRUN if some kernel wrote past the end of a buffer
 * (tsdp_last_error names its size).  *h_checked (may be null) receives the number of buffers verified.
 * Errors: ARG, CUDA, OVERRUN. */
int tsdp_debug_check_guards(tsdp_ctx* ctx, int* h_checked);

/* Exercise the time-out path of the tensor-core GEMM without hanging anything (test interface, precision 1).  Every
 * wait inside the kernel is bounded; normally the bound (about a second) is never reached.  After this call the NEXT
 * tsdp_gemm launch runs with the bound set to `wait_cycles` SM clock cycles (1e3 .. 2e9) and with one operand tile
 * withheld from CTA 0: that CTA's waits run out, it records TSDP_ERR_TIMEOUT, drains its copies, frees its tensor
 * memory and returns, while the other CTAs finish normally.  tsdp_gemm then returns TSDP_ERR_TIMEOUT (its output is
 * incomplete), the status word is cleared, and the context stays usable.  One-shot.  Errors: ARG. */
int tsdp_debug_arm_gemm_timeout(tsdp_ctx* ctx, long long wait_cycles);

/* The same GEMM launched `reps` times back to back between one pair of CUDA events on `cuda_stream`
 * (after one untimed launch); *h_ms (HOST) receives the mean device time of one launch in milliseconds.
 * With EPI 2 the output accumulates over the launches.  Measurement interface; synchronous. */
int tsdp_gemm_timed(tsdp_ctx* ctx, const void* d_A, const void* d_W, const float* d_bias, int M, int N, int K,
                    int epi, void* d_out, int reps, float* h_ms, void* cuda_stream);

/* Per-request efficiency counters of the last tsdp_sample_chunk / tsdp_sample_chunk_host / tsdp_serve /
 * tsdp_round call (zeroed when that call starts): h_counts [n, 4] int32 on the HOST, per request
 * {n_draft: drafts proposed, n_accept: drafts accepted, rounds, n_diffusion: reverse steps taken
 * (= T once the chunk is complete)}.  n <= the number of requests of that call.  Synchronises the
 * device.  Errors: ARG, CUDA. */
int tsdp_request_counts(tsdp_ctx* ctx, int* h_counts, int n);
/* Intermediate ("process") reward of the scheduler's training signal (Sec. 3.3, "Reward function"),
 * one value per request of the last call, computed on the device from the counters above:
 *     r = (n_accept / n_draft + n_accept / n_diffusion) * lambda,
 *     lambda = (R_final / 4) / ceil(T_max / dt),
 * T_max the task's step limit and dt the number of task steps between scheduler updates.  A ratio
 * whose denominator is zero counts 0.  h_reward [n] fp32 on the HOST.  The final (success / failure)
 * reward needs the simulator and is the caller's.  Errors: ARG (n, T_max < 1, dt < 1), CUDA. */
int tsdp_process_reward(tsdp_ctx* ctx, float R_final, int T_max, int dt, float* h_reward, int n);

/* Distillation objective of the drafter against the frozen base model (Sec. 3.2, "Draft model"), forward
 * evaluation only (no parameter update: training is outside this library).  For sample n < N (<= max_B) the
 * clean chunk d_x0[n] ([N, H, A] DEVICE) is noised at a timestep t_n = floor(T u_n) with Gaussian noise eps_n,
 * both from the counter-based generator (u_n: the uniform of (seed, n, timestep code 0); eps_n: the initial-latent
 * normals of (seed, n)):  x_t = sqrt(abar_t) x0 + sqrt(1 - abar_t) eps.  Both networks are run on (x_t, t_n,
 * d_obs[n]) and
 *     L_pred = mean_n |m^ - m|^2                       (m, m^: outputs of base and drafter; norm over H*A),
 *     L_norm = mean over samples with t_n >= 1 of |(mu^ - mu) / sigma_t|^2   (posterior means; sigma_0 = 0),
 *     L      = lambda1 L_pred + lambda2 L_norm.
 * h_out[4] (HOST, double) = {L_pred, L_norm, L, mean over t_n >= 1 of 2 Phi(-|d|/2)}; the last value is the
 * probability that the acceptance test of Sec. 3.1 takes a draft whose mean is off by d = (mu^ - mu)/sigma_t.
 * Uses the round's work buffers: call between chunks.  Synchronous.  Errors: ARG (N, null pointers, a
 * TSDP_ARCH_FROZEN drafter), STATE (weights not loaded), TOO_LARGE, CUDA. */
int tsdp_distill_loss(tsdp_ctx* ctx, const float* d_x0, const float* d_obs, int N, uint64_t seed, float lambda1,
                      float lambda2, double* h_out);

/* One gradient step of that objective on the drafter, the base model frozen (Sec. 3.2, "Draft Model Training": only
 * the drafter's parameters are updated).  Built for the closed-form Gaussian drafter (draft.arch = TSDP_ARCH_GAUSS,
 * parameters theta = (m0, s0), m^(x, t) = sqrt(1 - abar)(x - sqrt(abar) m0) / (abar s0^2 + 1 - abar)), whose gradient
 * is analytic; the base model may be any architecture.  Same draws (t_n, eps_n) as tsdp_distill_loss.  On the device:
 * noising, the base forward, the per-sample gradient terms, their reduction and  theta <- theta - lr dL/dtheta.
 * h_out[7] (HOST, double) = {L_pred, L_norm, L (all before the step), dL/dm0, dL/ds0, m0, s0 after the step}.
 * The new parameters are in force for every later call (rounds captured in graphs are captured again).  lr = 0
 * evaluates the gradient only.  Backward passes through the transformer / UNet drafters are not built.
 * Uses the round's work buffers: call between chunks.  Synchronous.
 * Errors: ARG (N, null pointers, a drafter that is not TSDP_ARCH_GAUSS, clip > 0, lr < 0), STATE, CUDA. */
int tsdp_distill_step(tsdp_ctx* ctx, const float* d_x0, const float* d_obs, int N, uint64_t seed, float lambda1,
                      float lambda2, float lr, double* h_out);

/* Copy the counters accumulated since the last reset (synchronises the device). */
int tsdp_stats(tsdp_ctx* ctx, tsdp_stats_t* out);
int tsdp_reset_stats(tsdp_ctx* ctx);
/* Number of kernels this library launched (or replayed through graphs) since the last reset. */
uint64_t tsdp_kernel_launches(const tsdp_ctx* ctx);


/* Per-kernel-family device timing with CUDA events, for the roofline report.  While enabled, rounds
 * are issued as plain launches (no graph) with an event pair around each launch on the caller's
 * stream.  Families: 0 GEMMs of the base model (tcgen05 or check-mode), 1 LayerNorm, 2 attention,
 * 3 embed/head/memory tokens, 4 draft-step kernel, 5 MLP / Gaussian denoiser, 6 GEMMs
 * of the drafter, 7 the persistent cluster drafter, 8 the fused
 * acceptance / commit kernel, 9 the cluster kernel as verifier, 10 / 11 / 12 the drafter's LayerNorm / attention /
 * embedding-head kernels (families 1-3 hold the base model's only).  A GEMM's flops count the rows it really
 * processed (the live candidates of the round's plan).  tsdp_profile(ctx, 0|1)
 * clears the record.  tsdp_profile_read fills three arrays of TSDP_PROF_FAMILIES entries: summed
 * milliseconds, summed algorithmic flops (2*M*N*K per GEMM launch, 0 elsewhere) and launch counts. */
enum { TSDP_PROF_FAMILIES = 13 };
int tsdp_profile(tsdp_ctx* ctx, int enable);
int tsdp_profile_read(tsdp_ctx* ctx, double* ms, double* flop, uint64_t* launches);

/* Verification tail without any allocation.  (The paper has no counterpart: this entry point exists
 * for integration, not for the method.)
 *
 * Who needs it: code that runs where device memory cannot be requested -- a control loop that was
 * handed a fixed memory budget at start-up, a plug-in inside a host application that owns the
 * allocator, a real-time thread that must not take the driver's allocation lock.  Such a caller
 * cannot create a tsdp_ctx (tsdp_init allocates), but it may already hold the candidate latents,
 * drafter means and base outputs of a round and only need the decision: the posterior mean of every
 * candidate, the log acceptance ratios, the first rejected step j*, and the committed latent
 * (reflection at j*, bonus step, or last draft).  This function does exactly what the fused
 * acceptance kernel of tsdp_sample_chunk does, on caller-owned buffers, and calls neither
 * cudaMalloc / cudaFree nor any routine that allocates.
 *
 * Its working memory (DDPM tables for T steps, t[B], j*[B], the counters, seed and round
 * parameters: under 64 KiB) is a fixed array inside the library image; every GPU that loads the
 * library holds it until the process exits.  Capacity: B <= TSDP_STATIC_MAX_B, T <= TSDP_STATIC_MAX_T,
 * K <= TSDP_MAX_K; larger sizes return TSDP_ERR_TOO_LARGE and print the limits to stderr.
 * The first call on a device looks up the array's device address.  Every call copies its small
 * inputs to the device, reads the results back and waits for `cuda_stream`, so it must not be made
 * while that stream is being captured into a graph.  All calls share the one array, which still holds the previous call's
 * values on entry (the function clears what must start at zero itself); two calls whose GPU work
 * overlaps -- different streams or threads -- race on it.  Synchronous: returns after `cuda_stream`
 * has finished the work.
 *
 *   device              CUDA device ordinal (made current)
 *   T, beta0, beta1, clip   DDPM schedule, as in tsdp_config_t
 *   d_xt   [B, K+1, D]  DEVICE, in/out: candidate latents, slot 0 = the round's input latent; on return
 *                       slot 0 of every unfinished environment holds the committed latent
 *   d_muhat [B, K, D]   DEVICE, in: drafter means (may be null when K = 0)
 *   d_eps  [B, K+1, D]  DEVICE, in: base-model outputs for every candidate
 *   h_t    [B]          HOST, in: timestep of each environment's input latent (-1 = finished, skipped)
 *   accept, seed        as in tsdp_sample_chunk; draft_nfe is ignored by the decision
 *   d_actions [B, D]    DEVICE, out: written for environments that reach t = -1 in this round
 *   h_t_new, h_jstar [B] HOST, out: new timesteps; first rejected step (K_eff+1 if none, -1 if finished)
 *   d_logalpha [B, K]   DEVICE, out, may be null
 * Errors: ARG, TOO_LARGE, CUDA (text on stderr). */
enum { TSDP_STATIC_MAX_B = 1024, TSDP_STATIC_MAX_T = 1024 };
int tsdp_verify_commit_static(int device, int T, float beta0, float beta1, float clip, float* d_xt,
                              const float* d_muhat, const float* d_eps, const int* h_t, int B, int K, int D,
                              const tsdp_accept_t* accept, uint64_t seed, float draft_nfe, float* d_actions,
                              int* h_t_new, int* h_jstar, float* d_logalpha, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* TSDP_H */
