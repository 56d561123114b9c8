"""GPU parity, kernel level: the tcgen05 GEMM and each denoiser against the fp64 oracle."""
import numpy as np
import pytest
import torch

from paper_2512_15773_b200 import binding, inputs
from oracle import nets as onets
from tests import helpers as hp

pytestmark = pytest.mark.gpu


def _gemm_case(smp, M, N, K, epi, rng):
    A = inputs.bf16_round(rng.normal(size=(M, K)))
    W = inputs.bf16_round(rng.normal(size=(N, K)) / np.sqrt(K))
    bias = rng.normal(size=N).astype(np.float32)
    dA = torch.tensor(A, dtype=torch.bfloat16, device="cuda")
    dW = torch.tensor(W, dtype=torch.bfloat16, device="cuda")
    db = torch.tensor(bias, device="cuda")
    ref = A @ W.T + bias.astype(np.float64)
    if epi == 1:
        ref = onets.gelu_tanh(ref)
    if epi in (0, 1):
        out = torch.zeros(M, N, dtype=torch.bfloat16, device="cuda")
    else:
        base = rng.normal(size=(M, N)).astype(np.float32)
        out = torch.tensor(base, device="cuda") if epi == 2 else torch.zeros(M, N, device="cuda")
        if epi == 2:
            ref = ref + base
    smp.gemm(dA, dW, db, M, N, K, epi, out)
    got = out.float().cpu().numpy().astype(np.float64)
    tol = 1e-2 if epi in (0, 1) else 2e-5          # bf16 output rounding vs fp32 accumulate only
    err = hp.max_rel(got, ref)
    assert err < tol, (M, N, K, epi, err)


def test_tcgen05_gemm_against_fp64():
    wl = hp.small_xfmr_workload(1)
    smp, *_ = hp.setup(wl, max_B=1, max_K=1)
    rng = np.random.default_rng(0)
    # every tile width (32/64/128/256 are picked from M and N), ragged M, multi-wave, long K
    for (M, N, K) in [(16, 128, 128), (144, 768, 256), (100, 32, 64), (129, 64, 512), (1000, 256, 128),
                      (2500, 384, 128), (19000, 256, 256), (40000, 512, 512), (4111, 128, 2048)]:
        for epi in (0, 1, 2, 3):
            _gemm_case(smp, M, N, K, epi, rng)
    smp.close()


@pytest.mark.parametrize("arch", ["mlp", "gauss"])
def test_small_denoisers(arch):
    rng = np.random.default_rng(1)
    if arch == "mlp":
        wl = dict(inputs.WORKLOADS["toy_mlp"])
    else:
        wl = dict(H=4, A=3, To=0, Do=0, T=100, precision=0, base=dict(arch="gauss"), draft=dict(arch="gauss"),
                  base_params=inputs.make_gauss_params(0.7, 0.5), draft_params=inputs.make_gauss_params(0.9, 0.4))
    N = 37
    smp, S, base, draft = hp.setup(wl, max_B=N, max_K=2)
    x = rng.normal(size=(N, wl["H"], wl["A"])).astype(np.float32)
    tau = rng.integers(0, 100, size=N).astype(np.int32); tau[0], tau[1] = 0, 99
    obs = inputs.make_obs(0, N, wl["To"], wl["Do"]) if wl["To"] else np.zeros((N, 0, 0))
    dx = torch.tensor(x, device="cuda"); dobs = torch.tensor(obs, dtype=torch.float32, device="cuda")
    for which, net in ((binding.BASE, base), (binding.DRAFT, draft)):
        out = torch.zeros_like(dx)
        smp.denoise(which, dx, tau, dobs if wl["To"] else None, N, out)
        ref = np.stack([net(x[n].astype(np.float64), int(tau[n]), obs[n]) for n in range(N)])
        assert hp.max_rel(out.cpu().numpy(), ref) < 1e-4
    smp.close()


def _transformer_case(precision, tol, shape):
    rng = np.random.default_rng(2)
    if shape == "small":
        wl = hp.small_xfmr_workload(precision, d=128, heads=4, layers=2, dd=256, dlayers=1, H=7, A=3, To=3, Do=5,
                                    gamma=1.0)
    elif shape == "long":
        # 50 tokens: four 16-query tiles with a ragged last one; head widths 128 and 96 (the latter takes the one-warp-per-row cross-attention)
        wl = hp.small_xfmr_workload(precision, d=256, heads=2, layers=2, dd=384, dlayers=1, H=50, A=3, To=3, Do=6,
                                    gamma=1.0)
        wl["draft"]["heads"] = 4
    elif shape == "no_obs":
        # the time token is the only memory token; widths 512 (8 heads) and 128 (2 heads)
        wl = hp.small_xfmr_workload(precision, d=512, heads=8, layers=1, dd=128, dlayers=2, H=16, A=4, To=0, Do=1,
                                    gamma=1.0)
        wl["draft"]["heads"] = 2
    elif shape == "one_obs":
        wl = hp.small_xfmr_workload(precision, d=512, heads=8, layers=2, dd=256, dlayers=1, H=11, A=2, To=1, Do=9,
                                    gamma=1.0)
        wl["draft"]["heads"] = 8
    else:
        wl = dict(inputs.WORKLOADS["pusht_xfmr"], precision=precision, gamma=1.0)
    N = 19      # 19*H token rows: ragged against the 128-row tiles
    smp, S, base, draft = hp.setup(wl, max_B=N, max_K=1)
    x = rng.normal(size=(N, wl["H"], wl["A"])).astype(np.float32)
    tau = rng.integers(0, 100, size=N).astype(np.int32); tau[0], tau[1] = 0, 99
    obs = inputs.make_obs(5, N, wl["To"], wl["Do"]) if wl["To"] else np.zeros((N, 0, wl["Do"]))
    dx = torch.tensor(x, device="cuda"); dobs = torch.tensor(obs, dtype=torch.float32, device="cuda")
    for which, net in ((binding.BASE, base), (binding.DRAFT, draft)):
        out = torch.zeros_like(dx)
        smp.denoise(which, dx, tau, dobs if wl["To"] else None, N, out)
        ref = np.stack([net(x[n].astype(np.float64), int(tau[n]), obs[n]) for n in range(N)])
        err = hp.max_rel(out.cpu().numpy(), ref)
        assert err < tol, (which, err)
    smp.close()


@pytest.mark.parametrize("precision,tol", [(0, 1e-4), (1, 2e-2)])
@pytest.mark.parametrize("shape", ["small", "pusht", "long", "no_obs", "one_obs"])
def test_transformer_denoiser(precision, tol, shape):
    _transformer_case(precision, tol, shape)


@pytest.mark.parametrize("shape", ["small", "pusht", "one_obs"])
def test_transformer_denoiser_bf16_without_the_cross_attention_fold(shape, monkeypatch):
    """The bf16 forward with separate LayerNorm / query GEMM / attention / output GEMM kernels (what shapes outside the
    fold's limits run), selected by the environment variable the library reads when weights are loaded."""
    monkeypatch.setenv("TSDP_NO_FOLD", "1")
    _transformer_case(1, 2e-2, shape)


@pytest.mark.parametrize("precision,tol", [(0, 1e-4), (1, 2e-2)])
@pytest.mark.parametrize("shape", ["small", "wide", "tc"])
def test_dit_denoiser(precision, tol, shape, monkeypatch):
    """Adaptive-LayerNorm transformer against the oracle: gated residual epilogue, modulated LayerNorm,
    bidirectional self-attention, cross-attention to the context tokens."""
    rng = np.random.default_rng(3)
    if shape == "tc":
        monkeypatch.setenv("TSDP_TC_ATTN", "2")      # single-candidate groups too (the default keeps those on mma.sync)
    if shape == "small":
        # 7 tokens, 12 context tokens (not a multiple of 16: the scalar context attention), head width 32
        wl = dict(H=7, A=3, To=12, Do=5, T=100, precision=precision, gamma=1.0,
                  base=dict(arch="dit", layers=2, d=128, heads=4), draft=dict(arch="dit", layers=1, d=256, heads=2))
    elif shape == "wide":
        # 50 tokens, 48 context tokens (tensor-core context attention over a ragged 64-key chunk), head widths 64 / 128
        wl = dict(H=50, A=14, To=48, Do=24, T=100, precision=precision, gamma=1.0,
                  base=dict(arch="dit", layers=2, d=256, heads=4), draft=dict(arch="dit", layers=1, d=128, heads=1))
    else:
        # 64-wide heads and 96 context tokens: in bf16 the context attention runs on tcgen05 (S = Q K^T and O = P V in
        # tensor memory, one and a half 64-key atoms)
        wl = dict(H=50, A=14, To=96, Do=24, T=100, precision=precision, gamma=1.0,
                  base=dict(arch="dit", layers=2, d=256, heads=4), draft=dict(arch="dit", layers=1, d=512, heads=8))
    N = 9
    smp, S, base, draft = hp.setup(wl, max_B=N, max_K=1)
    x = rng.normal(size=(N, wl["H"], wl["A"])).astype(np.float32)
    tau = rng.integers(0, 100, size=N).astype(np.int32); tau[0], tau[1] = 0, 99
    obs = inputs.make_obs(5, N, wl["To"], wl["Do"])
    dx = torch.tensor(x, device="cuda"); dobs = torch.tensor(obs, dtype=torch.float32, device="cuda")
    for which, net in ((binding.BASE, base), (binding.DRAFT, draft)):
        out = torch.zeros_like(dx)
        smp.denoise(which, dx, tau, dobs, N, out)
        ref = np.stack([net(x[n].astype(np.float64), int(tau[n]), obs[n]) for n in range(N)])
        err = hp.max_rel(out.cpu().numpy(), ref)
        assert err < tol, (which, err)
    smp.close()


@pytest.mark.parametrize("precision,tol", [(0, 1e-4), (1, 2e-2)])
@pytest.mark.parametrize("shape", ["two_levels", "three_levels"])
def test_unet_denoiser(precision, tol, shape):
    """1-D conv UNet against the oracle: convolutions as GEMMs over the zero-padded layout (tensor-core
    path in precision 1), GroupNorm + Mish + FiLM, pooling, repetition, skip concatenation, 1x1 residuals."""
    rng = np.random.default_rng(4)
    if shape == "two_levels":
        wl = dict(H=8, A=3, To=2, Do=12, T=100, precision=precision, gamma=1.0,
                  base=dict(arch="unet", layers=2, d=128, heads=8, temb=32), draft=dict(arch="unet", layers=1, d=128, heads=4, temb=16))
    else:
        wl = dict(H=16, A=10, To=2, Do=24, T=100, precision=precision, gamma=1.0,
                  base=dict(arch="unet", layers=3, d=128, heads=8, temb=64), draft=dict(arch="xfmr", layers=1, d=128, heads=4))
    N = 11      # 11 * 20 padded rows: ragged against the 128-row tiles
    smp, S, base, draft = hp.setup(wl, max_B=N, max_K=1)
    x = rng.normal(size=(N, wl["H"], wl["A"])).astype(np.float32)
    tau = rng.integers(0, 100, size=N).astype(np.int32); tau[0], tau[1] = 0, 99
    obs = inputs.make_obs(5, N, wl["To"], wl["Do"])
    dx = torch.tensor(x, device="cuda"); dobs = torch.tensor(obs, dtype=torch.float32, device="cuda")
    for which, net in ((binding.BASE, base), (binding.DRAFT, draft)):
        out = torch.zeros_like(dx)
        smp.denoise(which, dx, tau, dobs, N, out)
        ref = np.stack([net(x[n].astype(np.float64), int(tau[n]), obs[n]) for n in range(N)])
        err = hp.max_rel(out.cpu().numpy(), ref)
        assert err < tol, (which, err)
    # a second call must give the same answer: the padding rows of every buffer are still zero
    out2 = torch.zeros_like(dx)
    smp.denoise(binding.BASE, dx, tau, dobs, N, out2)
    ref = np.stack([base(x[n].astype(np.float64), int(tau[n]), obs[n]) for n in range(N)])
    assert hp.max_rel(out2.cpu().numpy(), ref) < tol
    smp.close()


def test_unet_split_reduction_is_reproducible_and_matches_the_unsplit_sums(monkeypatch):
    """At small batch the convolution GEMMs cut their reduction into parts that run on otherwise idle SMs; the
    GroupNorm kernel adds the partial sums in a fixed order.  So two runs must agree bit for bit, and against the
    same forward with the split switched off (other summation order) the difference must stay at rounding level."""
    wl = dict(H=16, A=10, To=2, Do=24, T=100, precision=1, gamma=1.0,
              base=dict(arch="unet", layers=3, d=128, heads=8, temb=64), draft=dict(arch="xfmr", layers=1, d=128, heads=4))
    rng = np.random.default_rng(9)
    N = 3
    x = rng.normal(size=(N, wl["H"], wl["A"])).astype(np.float32)
    tau = np.array([5, 50, 99], dtype=np.int32)
    obs = inputs.make_obs(6, N, wl["To"], wl["Do"])
    outs = []
    for split in (True, True, False):
        if split:
            monkeypatch.delenv("TSDP_NO_KSPLIT", raising=False)
        else:
            monkeypatch.setenv("TSDP_NO_KSPLIT", "1")
        smp, S, base, draft = hp.setup(wl, max_B=N, max_K=1)
        dx = torch.tensor(x, device="cuda"); dobs = torch.tensor(obs, dtype=torch.float32, device="cuda")
        out = torch.zeros_like(dx)
        smp.denoise(binding.BASE, dx, tau, dobs, N, out)
        outs.append(out.cpu().numpy().copy())
        smp.close()
    assert np.array_equal(outs[0], outs[1])                       # same split, same bits
    ref = np.stack([base(x[n].astype(np.float64), int(tau[n]), obs[n]) for n in range(N)])
    assert hp.max_rel(outs[0], ref) < 2e-2 and hp.max_rel(outs[2], ref) < 2e-2
    assert hp.max_rel(outs[0], outs[2]) < 2e-2 and not np.array_equal(outs[0], outs[2])   # the split really was taken


def test_gemm_bounded_wait_runs_out_and_the_context_recovers():
    """Failure detection without a fault: one CTA of the tensor-core GEMM is starved of an operand tile (a barrier
    that nothing completes) with the wait limit lowered to about a millisecond.  The kernel must return by giving up
    its waits, the call must report TSDP_ERR_TIMEOUT, the status word must be cleared, and the next ordinary calls on
    the same context must pass their parity checks."""
    import time
    wl = hp.small_xfmr_workload(1)
    smp, *_ = hp.setup(wl, max_B=1, max_K=1)
    rng = np.random.default_rng(5)
    _gemm_case(smp, 4000, 512, 512, 0, rng)                       # healthy before
    M, N, K = 4000, 512, 512
    dA = torch.zeros(M, K, dtype=torch.bfloat16, device="cuda"); dW = torch.zeros(N, K, dtype=torch.bfloat16, device="cuda")
    out = torch.zeros(M, N, dtype=torch.bfloat16, device="cuda")
    smp.arm_gemm_timeout(2_000_000)                               # about 1 ms of SM clock
    t0 = time.perf_counter()
    with pytest.raises(binding.TsdpError) as e:
        smp.gemm(dA, dW, None, M, N, K, 0, out)
    assert e.value.status == 5                                    # TSDP_ERR_TIMEOUT
    assert time.perf_counter() - t0 < 5.0                         # gave up after milliseconds, not after the default second per wait
    # one-shot and cleared: the same context works again, every epilogue
    for epi in (0, 1, 2, 3):
        _gemm_case(smp, 4000, 512, 512, epi, rng)
    _gemm_case(smp, 129, 64, 512, 2, rng)
    with pytest.raises(binding.TsdpError):
        smp.arm_gemm_timeout(10)                                  # below the accepted range
    smp.close()


def test_fused_qkv_attention_equals_the_separate_kernels(monkeypatch):
    """With 64-wide heads and 16-token chunks the QKV projection and the causal self-attention are one tensor-core
    kernel (the attention runs in the GEMM's epilogue on the tile it has just produced).  It shares the attention
    arithmetic with the stand-alone kernel, so the denoiser output must be bit-identical with the fusion switched off;
    both are then held to the oracle.  301 candidates: 37 full 128-row tiles and a ragged one."""
    wl = dict(inputs.WORKLOADS["pusht_xfmr"], precision=1, gamma=1.0)
    N = 301
    rng = np.random.default_rng(4)
    x = rng.normal(size=(N, wl["H"], wl["A"])).astype(np.float32)
    tau = rng.integers(0, 100, size=N).astype(np.int32)
    obs = inputs.make_obs(6, N, wl["To"], wl["Do"])
    outs = []
    for fused in (True, False):
        if not fused:
            monkeypatch.setenv("TSDP_NO_FUSED_ATTN", "1")
        smp, S, base, draft = hp.setup(wl, max_B=N, max_K=1)
        dx = torch.tensor(x, device="cuda"); dobs = torch.tensor(obs, dtype=torch.float32, device="cuda")
        out = torch.zeros_like(dx)
        smp.denoise(binding.BASE, dx, tau, dobs, N, out)
        outs.append(out.clone())
        if fused:
            got = out.cpu().numpy()
            for n in (0, 7, 8, 127, 300):
                ref = base(x[n].astype(np.float64), int(tau[n]), obs[n])
                assert hp.max_rel(got[n], ref) < 2e-2, n
        smp.close()
    assert torch.equal(outs[0], outs[1])


def test_fused_qkv_attention_kernel_against_fp64():
    """tsdp_gemm, epilogue 4: projection with head-major output features [Q_h | K_h | V_h] and the causal attention
    of every 16-row chunk, against the definition in fp64 (softmax(Q K^T / 8) V per head, q / k / v rounded to bf16
    as the kernel keeps them)."""
    wl = hp.small_xfmr_workload(1)
    smp, *_ = hp.setup(wl, max_B=1, max_K=1)
    rng = np.random.default_rng(7)
    for M, d in ((16, 64), (2000, 256), (6544, 512)):
        heads = d // 64
        A = inputs.bf16_round(rng.normal(size=(M, d)))
        W = inputs.bf16_round(rng.normal(size=(3 * d, d)) / np.sqrt(d))
        bias = rng.normal(size=3 * d).astype(np.float32)
        qkv = inputs.bf16_round(A @ W.T + bias.astype(np.float64)).reshape(M // 16, 16, heads, 3, 64)
        q, k, v = qkv[:, :, :, 0], qkv[:, :, :, 1], qkv[:, :, :, 2]                     # [chunk, token, head, 64]
        s = np.einsum("cihe,cjhe->chij", q, k) / 8.0
        s = np.where(np.tril(np.ones((16, 16), dtype=bool)), s, -np.inf)
        p = np.exp(s - s.max(-1, keepdims=True)); p /= p.sum(-1, keepdims=True)
        ref = np.einsum("chij,cjhe->cihe", p, v).reshape(M, d)
        out = torch.zeros(M, d, dtype=torch.bfloat16, device="cuda")
        smp.gemm(torch.tensor(A, dtype=torch.bfloat16, device="cuda"), torch.tensor(W, dtype=torch.bfloat16, device="cuda"),
                 torch.tensor(bias, device="cuda"), M, 3 * d, d, 4, out)
        assert hp.max_rel(out.float().cpu().numpy().astype(np.float64), ref) < 1.5e-2, (M, d)
    smp.close()


def test_gemm_pair_form_gives_the_same_bits_as_the_single_cta_form(monkeypatch):
    """The two-CTA form of the tensor-core GEMM (tcgen05 cta_group::2: 256 x 256 tiles on clusters of two CTAs, each
    staging half of the W tile) accumulates every output element in the same order as the single-CTA form, so every
    epilogue must return identical bits; both are held to fp64 elsewhere.  Ragged M, odd and even numbers of
    128-row blocks, short and long reductions."""
    wl = hp.small_xfmr_workload(1)
    shapes = [(129, 256, 64), (1000, 512, 128), (5000, 256, 1024), (33000, 1024, 512), (8200, 768, 2048)]
    outs = {}
    for mode in ("0", "2"):
        monkeypatch.setenv("TSDP_GEMM_PAIR", mode)
        smp, *_ = hp.setup(wl, max_B=1, max_K=1)
        g = torch.Generator(device="cuda").manual_seed(3)
        res = []
        for (M, N, K) in shapes:
            A = torch.randn(M, K, device="cuda", generator=g).to(torch.bfloat16)
            W = (torch.randn(N, K, device="cuda", generator=g) / np.sqrt(K)).to(torch.bfloat16)
            bias = torch.randn(N, device="cuda", generator=g)
            for epi in (0, 1, 2, 3):
                out = (torch.zeros(M, N, dtype=torch.bfloat16, device="cuda") if epi in (0, 1)
                       else torch.full((M, N), 0.25, device="cuda"))
                smp.gemm(A, W, bias, M, N, K, epi, out)
                res.append(out.clone())
        outs[mode] = res
        smp.close()
    for a, b in zip(outs["0"], outs["2"]):
        assert torch.equal(a, b)
