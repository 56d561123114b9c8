"""ctypes binding of libtsdp.so: argument marshalling only -- every step of the speculative round
runs in the library's CUDA kernels.  There is no CPU fallback: loading fails loudly when the shared
library is missing, and tsdp_init fails when no CUDA device is present."""
import ctypes as C
import os

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libtsdp.so")

TSDP_MAX_T = 1024
ARCH = {"gauss": 0, "mlp": 1, "xfmr": 2, "dit": 3, "unet": 4, "frozen": 5}     # "frozen": drafter only, no weights
BASE, DRAFT, SCHED = 0, 1, 2
EXPORTS = ["tsdp_init", "tsdp_destroy", "tsdp_strerror", "tsdp_last_error", "tsdp_weights_count",
           "tsdp_load_weights", "tsdp_set_schedule", "tsdp_sample_chunk", "tsdp_sample_chunk_host",
           "tsdp_round", "tsdp_denoise", "tsdp_gemm", "tsdp_gemm_timed", "tsdp_stats", "tsdp_reset_stats",
           "tsdp_kernel_launches", "tsdp_profile", "tsdp_profile_read", "tsdp_verify_commit_static", "tsdp_set_scheduler", "tsdp_set_progress",
           "tsdp_sched_eval", "tsdp_serve", "tsdp_request_counts", "tsdp_process_reward", "tsdp_distill_loss", "tsdp_distill_step", "tsdp_debug_arm_gemm_timeout", "tsdp_debug_check_guards"]
PROF_FAMILIES = ["gemm", "layernorm", "attention", "embed_head", "round", "small_net", "gemm_draft", "drafter_cluster", "accept", "verifier_cluster",
                 "layernorm_draft", "attention_draft", "embed_head_draft"]


class NetT(C.Structure):
    _fields_ = [("arch", C.c_int), ("layers", C.c_int), ("d", C.c_int), ("heads", C.c_int), ("temb", C.c_int)]


class ConfigT(C.Structure):
    _fields_ = [("base", NetT), ("draft", NetT), ("H", C.c_int), ("A", C.c_int), ("obs_tokens", C.c_int),
                ("obs_dim", C.c_int), ("T", C.c_int), ("beta0", C.c_float), ("beta1", C.c_float),
                ("clip", C.c_float), ("max_B", C.c_int), ("max_K", C.c_int), ("precision", C.c_int),
                ("device", C.c_int), ("draft_nfe", C.c_float), ("use_graph", C.c_int), ("drafter", C.c_int), ("verifier", C.c_int)]


class AcceptT(C.Structure):
    _fields_ = [("mode", C.c_int), ("lam", C.c_float), ("sigma_scale", C.c_float), ("bonus", C.c_int)]


class StatsT(C.Structure):
    _fields_ = [("chunks", C.c_uint64), ("rounds", C.c_uint64), ("env_rounds", C.c_uint64),
                ("base_evals", C.c_uint64), ("draft_evals", C.c_uint64), ("drafts_tested", C.c_uint64),
                ("drafts_accepted", C.c_uint64), ("rejections", C.c_uint64), ("bonus_steps", C.c_uint64),
                ("steps_advanced", C.c_uint64), ("draft_rounds", C.c_uint64), ("nfe", C.c_double),
                ("hist_drafted", C.c_uint64 * TSDP_MAX_T), ("hist_tested", C.c_uint64 * TSDP_MAX_T),
                ("hist_accepted", C.c_uint64 * TSDP_MAX_T), ("call_ms_p50", C.c_double), ("call_ms_p99", C.c_double),
                ("call_ms_samples", C.c_uint64), ("cand_dense", C.c_uint64), ("cand_computed", C.c_uint64)]


class TsdpError(RuntimeError):
    def __init__(self, status, what, detail=""):
        self.status = status
        super().__init__(f"{what}: status {status} ({detail})")


_lib = None


def load_library():
    """dlopen libtsdp.so (built in-tree by paper_2512_15773_b200.build) and declare its prototypes."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: run `python -m paper_2512_15773_b200.build` "
                          "(there is no CPU fallback)")
    lib = C.CDLL(LIB_PATH)
    vp, i, u64, fp = C.c_void_p, C.c_int, C.c_uint64, C.c_void_p
    lib.tsdp_init.argtypes = [C.POINTER(ConfigT), C.POINTER(vp)]
    lib.tsdp_destroy.argtypes = [vp]; lib.tsdp_destroy.restype = None
    lib.tsdp_strerror.argtypes = [i]; lib.tsdp_strerror.restype = C.c_char_p
    lib.tsdp_last_error.argtypes = [vp]; lib.tsdp_last_error.restype = C.c_char_p
    lib.tsdp_weights_count.argtypes = [C.POINTER(ConfigT), i]; lib.tsdp_weights_count.restype = C.c_size_t
    lib.tsdp_load_weights.argtypes = [vp, i, fp, C.c_size_t]
    lib.tsdp_set_schedule.argtypes = [vp, C.POINTER(C.c_int), C.POINTER(AcceptT), i]
    lib.tsdp_sample_chunk.argtypes = [vp, fp, i, i, C.POINTER(AcceptT), u64, fp, vp]
    lib.tsdp_sample_chunk_host.argtypes = [vp, fp, i, i, C.POINTER(AcceptT), u64, fp]
    lib.tsdp_round.argtypes = [vp, fp, i, i, C.POINTER(AcceptT), u64, fp, fp, fp, fp, fp, fp, fp, vp]
    lib.tsdp_denoise.argtypes = [vp, i, fp, fp, fp, i, fp, vp]
    lib.tsdp_gemm.argtypes = [vp, fp, fp, fp, i, i, i, i, fp, vp]
    lib.tsdp_gemm_timed.argtypes = [vp, fp, fp, fp, i, i, i, i, fp, i, C.POINTER(C.c_float), vp]
    lib.tsdp_verify_commit_static.argtypes = [i, i, C.c_float, C.c_float, C.c_float, fp, fp, fp, fp, i, i, i,
                                              C.POINTER(AcceptT), u64, C.c_float, fp, fp, fp, fp, vp]
    lib.tsdp_serve.argtypes = [vp, fp, i, i, i, C.POINTER(AcceptT), u64, fp, vp]
    lib.tsdp_set_scheduler.argtypes = [vp, i]
    lib.tsdp_set_progress.argtypes = [vp, fp, i]
    lib.tsdp_sched_eval.argtypes = [vp, fp, fp, fp, i, fp, vp]
    lib.tsdp_request_counts.argtypes = [vp, vp, i]
    lib.tsdp_distill_loss.argtypes = [vp, fp, fp, i, u64, C.c_float, C.c_float, vp]
    lib.tsdp_distill_step.argtypes = [vp, fp, fp, i, u64, C.c_float, C.c_float, C.c_float, vp]
    lib.tsdp_debug_arm_gemm_timeout.argtypes = [vp, C.c_longlong]
    lib.tsdp_debug_check_guards.argtypes = [vp, C.POINTER(C.c_int)]
    lib.tsdp_process_reward.argtypes = [vp, C.c_float, i, i, fp, i]
    lib.tsdp_stats.argtypes = [vp, C.POINTER(StatsT)]
    lib.tsdp_reset_stats.argtypes = [vp]
    lib.tsdp_kernel_launches.argtypes = [vp]; lib.tsdp_kernel_launches.restype = u64
    lib.tsdp_profile.argtypes = [vp, i]
    lib.tsdp_profile_read.argtypes = [vp, fp, fp, fp]
    _lib = lib
    return lib


def make_config(H, A, To, Do, base, draft, T=100, beta0=1e-4, beta1=0.02, clip=0.0, max_B=1, max_K=8,
                precision=1, device=0, draft_nfe=0.0, use_graph=1, drafter=0, verifier=0):
    def net(n):
        return NetT(ARCH[n["arch"]], n.get("layers", 0), n.get("d", n.get("width", 0)), n.get("heads", 0),
                    n.get("temb", 32))
    return ConfigT(net(base), net(draft), H, A, To, Do, T, beta0, beta1, clip, max_B, max_K, precision, device,
                   draft_nfe, use_graph, drafter, verifier)


def pack_weights(p):
    """Flatten a parameter dict (the layout the input generators produce) into the fp32 blob order
    documented in tsdp.h."""
    a = p["arch"]
    if a == "gauss":
        parts = [[p["m0"], p["s0"]]]
    elif a == "mlp":
        parts = []
        for W, b in zip(p["W"], p["b"]):
            parts += [W, b]
    elif a == "unet":
        parts = [p[k] for k in ("W_in", "b_in", "Wt1", "bt1", "Wt2", "bt2")]
        for R in p["blocks"]:
            parts += [R[k] for k in ("W1", "b1", "g1", "be1", "Wf", "bf", "W2", "b2", "g2", "be2")]
            if "Wr" in R:
                parts += [R["Wr"], R["br"]]
        parts += [p[k] for k in ("Wh", "bh", "gh", "beh", "W_out", "b_out")]
    elif a == "dit":
        parts = [p[k] for k in ("W_in", "b_in", "pos", "W_ctx", "b_ctx", "cpos", "Wt1", "bt1", "Wt2", "bt2")]
        for L in p["layers"]:
            parts += [L[k] for k in ("Wmod", "bmod", "Wqkv", "bqkv", "Wo", "bo", "lnc_g", "lnc_b", "Wq2", "bq2", "Wkv2", "bkv2",
                                     "Wo2", "bo2", "W1", "b1", "W2", "b2")]
        parts += [p["Wmodf"], p["bmodf"], p["W_out"], p["b_out"]]
    elif a == "sched":
        parts = [p[k] for k in ("W_o", "b_o", "W_a", "b_a", "W_p", "b_p", "W_1", "b_1", "W_2", "b_2")]
    elif a == "xfmr":
        parts = [p["W_in"], p["b_in"], p["pos"], p["W_obs"], p["b_obs"], p["cpos"]]
        for L in p["layers"]:
            parts += [L[k] for k in ("ln1_g", "ln1_b", "Wqkv", "bqkv", "Wo", "bo", "ln2_g", "ln2_b", "Wq2", "bq2",
                                     "Wkv2", "bkv2", "Wo2", "bo2", "ln3_g", "ln3_b", "W1", "b1", "W2", "b2")]
        parts += [p["lnf_g"], p["lnf_b"], p["W_out"], p["b_out"]]
    else:
        raise ValueError(a)
    return np.concatenate([np.asarray(x, dtype=np.float32).reshape(-1) for x in parts])


def _ptr(t):
    """Device or host address of a torch tensor / numpy array / None."""
    if t is None:
        return None
    if isinstance(t, np.ndarray):
        return t.ctypes.data
    return t.data_ptr()


def verify_commit_static(d_xt, d_muhat, d_eps, h_t, B, K, D, accept, seed, d_actions, h_t_new, h_jstar,
                         d_logalpha=None, T=100, beta0=1e-4, beta1=0.02, clip=0.0, device=0, stream=0):
    """tsdp_verify_commit_static: the fused acceptance / commit step on caller-owned buffers, for
    callers that may not allocate device memory (no context, no workspace; see tsdp.h)."""
    lib = load_library()
    st = lib.tsdp_verify_commit_static(device, T, beta0, beta1, clip, _ptr(d_xt), _ptr(d_muhat), _ptr(d_eps),
                                       _ptr(h_t), B, K, D, C.byref(accept), seed, 0.0, _ptr(d_actions),
                                       _ptr(h_t_new), _ptr(h_jstar), _ptr(d_logalpha), stream)
    if st != 0:
        raise TsdpError(st, "tsdp_verify_commit_static", lib.tsdp_strerror(st).decode())


class Sampler:
    """Thin owner of a tsdp_ctx.  Tensors passed in must be contiguous and of the documented dtype;
    torch is used by callers only to own device memory and streams."""

    def __init__(self, cfg):
        self.lib = load_library()
        self.cfg = cfg
        self.D = cfg.H * cfg.A
        h = C.c_void_p()
        st = self.lib.tsdp_init(C.byref(cfg), C.byref(h))
        if st != 0:
            raise TsdpError(st, "tsdp_init", self.lib.tsdp_strerror(st).decode())
        self.h = h

    def close(self):
        if getattr(self, "h", None):
            self.lib.tsdp_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, st, what):
        if st != 0:
            raise TsdpError(st, what, self.lib.tsdp_strerror(st).decode() + "; " +
                            self.lib.tsdp_last_error(self.h).decode())

    def weights_count(self, which):
        return self.lib.tsdp_weights_count(C.byref(self.cfg), which)

    def load_weights(self, which, params_or_blob):
        blob = params_or_blob if isinstance(params_or_blob, np.ndarray) else pack_weights(params_or_blob)
        blob = np.ascontiguousarray(blob, dtype=np.float32)
        self._check(self.lib.tsdp_load_weights(self.h, which, blob.ctypes.data, blob.size), "tsdp_load_weights")

    def set_schedule(self, Ks, accepts):
        n = len(Ks)
        if n == 0:
            self._check(self.lib.tsdp_set_schedule(self.h, None, None, 0), "tsdp_set_schedule")
            return
        ka = (C.c_int * n)(*Ks)
        aa = (AcceptT * n)(*accepts)
        self._check(self.lib.tsdp_set_schedule(self.h, ka, aa, n), "tsdp_set_schedule")

    def set_scheduler(self, enable):
        self._check(self.lib.tsdp_set_scheduler(self.h, int(enable)), "tsdp_set_scheduler")

    def set_progress(self, h_progress):
        a = np.ascontiguousarray(h_progress, dtype=np.float32)
        self._check(self.lib.tsdp_set_progress(self.h, a.ctypes.data, a.size), "tsdp_set_progress")

    def sched_eval(self, d_obs, d_prev_actions, h_progress, B):
        prog = np.ascontiguousarray(h_progress, dtype=np.float32)
        out = np.zeros((B, 8), dtype=np.float32)
        self._check(self.lib.tsdp_sched_eval(self.h, _ptr(d_obs), _ptr(d_prev_actions), prog.ctypes.data, B,
                                             out.ctypes.data, 0), "tsdp_sched_eval")
        return out

    def distill_loss(self, d_x0, d_obs, N, seed, lambda1=1.0, lambda2=1.0):
        """(L_pred, L_norm, L, mean acceptance probability) of the drafter against the base on N noised chunks."""
        out = np.zeros(4, dtype=np.float64)
        self._check(self.lib.tsdp_distill_loss(self.h, _ptr(d_x0), _ptr(d_obs), N, seed, lambda1, lambda2, out.ctypes.data),
                    "tsdp_distill_loss")
        return tuple(float(v) for v in out)

    def distill_step(self, d_x0, d_obs, N, seed, lambda1=1.0, lambda2=1.0, lr=0.1):
        """One gradient step on the Gaussian drafter: (L_pred, L_norm, L, dL/dm0, dL/ds0, m0', s0')."""
        out = np.zeros(7, dtype=np.float64)
        self._check(self.lib.tsdp_distill_step(self.h, _ptr(d_x0), _ptr(d_obs), N, seed, lambda1, lambda2, lr, out.ctypes.data),
                    "tsdp_distill_step")
        return tuple(float(v) for v in out)

    def request_counts(self, n):
        """[n, 4] int32 per request of the last call: drafts proposed, drafts accepted, rounds, reverse steps taken."""
        out = np.zeros((n, 4), dtype=np.int32)
        self._check(self.lib.tsdp_request_counts(self.h, out.ctypes.data, n), "tsdp_request_counts")
        return out

    def process_reward(self, R_final, T_max, dt, n):
        out = np.zeros(n, dtype=np.float32)
        self._check(self.lib.tsdp_process_reward(self.h, R_final, T_max, dt, out.ctypes.data, n), "tsdp_process_reward")
        return out

    def sample_chunk(self, d_obs, B, K, accept, seed, d_actions, stream=0):
        self._check(self.lib.tsdp_sample_chunk(self.h, _ptr(d_obs), B, K, C.byref(accept), seed, _ptr(d_actions),
                                               stream), "tsdp_sample_chunk")

    def serve(self, d_obs, N, slots, K, accept, seed, d_actions, stream=0):
        self._check(self.lib.tsdp_serve(self.h, _ptr(d_obs), N, slots, K, C.byref(accept), seed, _ptr(d_actions), stream),
                    "tsdp_serve")

    def sample_chunk_host(self, h_obs, B, K, accept, seed, h_actions):
        self._check(self.lib.tsdp_sample_chunk_host(self.h, _ptr(h_obs), B, K, C.byref(accept), seed,
                                                    _ptr(h_actions)), "tsdp_sample_chunk_host")

    def round(self, d_obs, B, K, accept, seed, d_x, h_t, d_xtilde=None, d_muhat=None, d_eps=None,
              d_logalpha=None, h_jstar=None, stream=0):
        self._check(self.lib.tsdp_round(self.h, _ptr(d_obs), B, K, C.byref(accept), seed, _ptr(d_x), _ptr(h_t),
                                        _ptr(d_xtilde), _ptr(d_muhat), _ptr(d_eps), _ptr(d_logalpha),
                                        _ptr(h_jstar), stream), "tsdp_round")

    def denoise(self, which, d_x, h_tau, d_obs, N, d_eps, stream=0):
        self._check(self.lib.tsdp_denoise(self.h, which, _ptr(d_x), _ptr(h_tau), _ptr(d_obs), N, _ptr(d_eps),
                                          stream), "tsdp_denoise")

    def gemm(self, d_A, d_W, d_bias, M, N, K, epi, d_out, stream=0):
        self._check(self.lib.tsdp_gemm(self.h, _ptr(d_A), _ptr(d_W), _ptr(d_bias), M, N, K, epi, _ptr(d_out),
                                       stream), "tsdp_gemm")

    def check_guards(self):
        """Verify the guard bytes behind every device buffer of the context; returns how many were checked."""
        n = C.c_int(0)
        self._check(self.lib.tsdp_debug_check_guards(self.h, C.byref(n)), "tsdp_debug_check_guards")
        return n.value

    def arm_gemm_timeout(self, wait_cycles):
        self._check(self.lib.tsdp_debug_arm_gemm_timeout(self.h, int(wait_cycles)), "tsdp_debug_arm_gemm_timeout")

    def gemm_timed(self, d_A, d_W, d_bias, M, N, K, epi, d_out, reps, stream=0):
        ms = C.c_float(0.0)
        self._check(self.lib.tsdp_gemm_timed(self.h, _ptr(d_A), _ptr(d_W), _ptr(d_bias), M, N, K, epi, _ptr(d_out),
                                             reps, C.byref(ms), stream), "tsdp_gemm_timed")
        return ms.value

    def stats(self):
        s = StatsT()
        self._check(self.lib.tsdp_stats(self.h, C.byref(s)), "tsdp_stats")
        T = self.cfg.T
        out = {k: getattr(s, k) for k, _ in StatsT._fields_ if not k.startswith("hist")}
        for k in ("hist_drafted", "hist_tested", "hist_accepted"):
            out[k] = np.array(getattr(s, k)[:T], dtype=np.int64)
        return out

    def reset_stats(self):
        self._check(self.lib.tsdp_reset_stats(self.h), "tsdp_reset_stats")

    def profile(self, enable):
        self._check(self.lib.tsdp_profile(self.h, int(enable)), "tsdp_profile")

    def profile_read(self):
        n = len(PROF_FAMILIES)
        ms, fl, ln = np.zeros(n), np.zeros(n), np.zeros(n, dtype=np.uint64)
        self._check(self.lib.tsdp_profile_read(self.h, ms.ctypes.data, fl.ctypes.data, ln.ctypes.data),
                    "tsdp_profile_read")
        return {f: dict(ms=float(ms[i]), flop=float(fl[i]), launches=int(ln[i])) for i, f in enumerate(PROF_FAMILIES)}

    def kernel_launches(self):
        return int(self.lib.tsdp_kernel_launches(self.h))
