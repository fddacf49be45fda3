"""Parity of the CUDA library (through the C ABI) with the fp64 oracle on seeded inputs."""
import numpy as np
import pytest
import torch

from paper_2510_25977_b200 import binding, inputs

import _gpu

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _gpu_ready():
    _gpu.require_gpu()


SKINNY, TENSOR = binding.FLAG_PATH_SKINNY, binding.FLAG_PATH_TENSOR


@pytest.mark.parametrize("flags", [0, SKINNY, TENSOR])
def test_cfg1_tiny_svd_config(oracle, flags):
    f = inputs.svd_factors(256, 688, 32, seed=0)
    X = inputs.activations(16, 256, seed=0)
    Y = _gpu.run_mlp(_gpu.factors_to_device(f), X.cuda(), flags=flags)
    _gpu.assert_close(Y, oracle.svdmlp(X, *f.tensors()), f"cfg1 flags={flags}")


@pytest.mark.parametrize("regs", [0, binding.FLAG_DECODE_REGISTERS])
@pytest.mark.parametrize("T", [1, 5, 8, 9, 16, 17, 33, 70])
def test_ragged_small_shapes_skinny(oracle, T, regs):
    """Both generations of the small-T kernels (TMA ring / register streaming) on ragged shapes."""
    f = inputs.direct_factors(264, 696, 40, seed=3, r_down=24)
    X = inputs.activations(T, 264, seed=3)
    Y = _gpu.run_mlp(_gpu.factors_to_device(f), X.cuda(), flags=SKINNY | regs)
    _gpu.assert_close(Y, oracle.svdmlp(X, *f.tensors()), f"ragged skinny T={T}")


def test_unequal_gate_up_ranks_run_on_skinny_path(oracle):
    f = inputs.direct_factors(128, 320, 16, seed=4)
    f2 = inputs.direct_factors(128, 320, 48, seed=5)
    mixed = inputs.Factors(128, 320, 16, 48, 16, f.Ug, f.Vg, f2.Uu, f2.Vu, f.Ud, f.Vd)
    X = inputs.activations(40, 128, seed=4)
    Y = _gpu.run_mlp(_gpu.factors_to_device(mixed), X.cuda())
    _gpu.assert_close(Y, oracle.svdmlp(X, *mixed.tensors()), "unequal ranks")


@pytest.mark.parametrize("pairs", [0, binding.FLAG_NO_TMEM_STRIP, binding.FLAG_NO_CTA_PAIRS])
@pytest.mark.parametrize("T", [33, 128, 130, 257, 600])
def test_ragged_shapes_tensor_path(oracle, T, pairs):
    """The tilings of the tcgen05 path (CTA pairs with the Z strip in tensor memory or in shared memory /
    single CTAs) on ragged shapes: Eq. 1 says the result does not depend on the blocking."""
    f = inputs.direct_factors(264, 696, 40, seed=6, r_down=24)
    X = inputs.activations(T, 264, seed=6)
    Y = _gpu.run_mlp(_gpu.factors_to_device(f), X.cuda(), flags=TENSOR | pairs)
    _gpu.assert_close(Y, oracle.svdmlp(X, *f.tensors()), f"ragged tensor T={T}")


@pytest.mark.parametrize("r", [64, 192, 256])
def test_tmem_strip_gateup_chunk_counts(oracle, r):
    """Gate/up with the Z strip in tensor memory: one, three (odd: the last ring slot of a branch holds a
    single K chunk) and four K chunks, several row strips per CTA pair, ragged T and ffn; the same shapes
    through the shared-memory-strip kernel must agree with the oracle as well."""
    d, ffn, T = 512, 1096, 900
    f = inputs.direct_factors(d, ffn, r, seed=11, r_down=64)
    X = inputs.activations(T, d, seed=11)
    ref = oracle.svdmlp(X, *f.tensors())
    fd = _gpu.factors_to_device(f)
    for flags in (TENSOR, TENSOR | binding.FLAG_NO_TMEM_STRIP):
        _gpu.assert_close(_gpu.run_mlp(fd, X.cuda(), flags=flags), ref, f"r={r} flags={flags:#x}")


@pytest.mark.parametrize("r", [320, 512])
def test_wide_rank_gateup_256_wide_tiles(oracle, r):
    """Ranks above 256: gate/up on 256 x 256 pair tiles (chosen when the tile count quantises well: here
    4 row-strip pairs x 37 column tiles = 2 rounds on 74 clusters) against the 128-wide tiling and the oracle;
    ragged T and ffn, five and eight K chunks."""
    d, ffn, T = 512, 9464, 1000
    f = inputs.direct_factors(d, ffn, r, seed=12, r_down=64, device="cuda")
    X = inputs.activations(T, d, seed=12, device="cuda")
    rows = inputs.sample_rows(T, max_rows=48)
    ref = _gpu.oracle_rows(oracle, f, X, rows)
    for flags in (TENSOR, TENSOR | binding.FLAG_NO_WIDE_GATEUP):
        Y = _gpu.run_mlp(f, X, flags=flags)
        _gpu.assert_close(Y[rows], ref, f"r={r} flags={flags:#x}")


@pytest.mark.parametrize("regs", [0, binding.FLAG_DECODE_REGISTERS])
@pytest.mark.parametrize("T", [1, 4, 8, 32])
def test_cfg2_decode(oracle, T, regs):
    f = inputs.direct_factors(4096, 11008, 256, seed=0, device="cuda")
    X = inputs.activations(T, 4096, seed=0, device="cuda")
    Y = _gpu.run_mlp(f, X, flags=regs)
    h = binding.svdmlp_create(*f.tensors(), max_T=T)
    assert binding.svdmlp_path_name(h, T) == "skinny"
    binding.svdmlp_destroy(h)
    _gpu.assert_close(Y, oracle.svdmlp(X, *f.tensors()), f"cfg2 T={T}")


@pytest.mark.parametrize("T", [512, 2048, 4096])
def test_cfg3_prefill_every_row(oracle, T):
    f = inputs.direct_factors(4096, 11008, 256, seed=0, device="cuda")
    X = inputs.activations(T, 4096, seed=0, device="cuda")
    h = binding.svdmlp_create(*f.tensors(), max_T=T)
    assert binding.svdmlp_path_name(h, T) == "tensor"
    Y = binding.svdmlp_forward(h, X)
    torch.cuda.synchronize()
    assert binding.svdmlp_last_device_status(h) == 0
    _gpu.assert_close(Y, oracle.svdmlp(X.cpu(), *(t.cpu() for t in f.tensors())), f"cfg3 T={T}")  # every row
    rows = inputs.sample_rows(T, max_rows=40)
    # rows are independent: a lone row gives the same answer through the small-T kernels
    Y1 = binding.svdmlp_forward(h, X[rows[3]:rows[3] + 1].contiguous())
    _gpu.assert_close(Y1, _gpu.oracle_rows(oracle, f, X, [rows[3]]), "single row")
    binding.svdmlp_destroy(h)


@pytest.mark.parametrize("r", [128, 512, 1024])
@pytest.mark.parametrize("T", [1, 8, 128, 2048, 8192])
def test_cfg4_rank_sweep(oracle, r, T):
    f = inputs.direct_factors(4096, 14336, r, seed=0, device="cuda")
    X = inputs.activations(T, 4096, seed=0, device="cuda")
    Y = _gpu.run_mlp(f, X)
    # every row up to T = 2048; at T = 8192 two rows of every 128-row tile (the oracle does a few hundred rows/s)
    rows = list(range(T)) if T <= 2048 else inputs.rows_of_every_tile(T, per_tile=2)
    _gpu.assert_close(Y[rows], _gpu.oracle_rows(oracle, f, X, rows), f"cfg4 r={r} T={T}")


@pytest.mark.parametrize("T,r,path", [(16, 1024, "skinny"), (24, 1024, "tensor"), (32, 1024, "tensor"), (32, 512, "skinny")])
def test_between_9_and_32_tokens_the_path_follows_the_decode_kernels_fit(oracle, T, r, path):
    """A handle made for at most 32 tokens: where the persistent decode kernel's shared-memory layout does not
    fit (ranks 1024 above 16 tokens) the tcgen05 kernels run, not the slower three-kernel fallback."""
    f = inputs.direct_factors(5120, 14336, r, seed=2, device="cuda")
    X = inputs.activations(T, 5120, seed=2, device="cuda")
    h = binding.svdmlp_create(*f.tensors(), max_T=T)
    try:
        assert binding.svdmlp_path_name(h, T) == path
        assert binding.svdmlp_path_name(h, 8) == "skinny"
        Y = binding.svdmlp_forward(h, X)
        torch.cuda.synchronize()
        assert binding.svdmlp_last_device_status(h) == 0
    finally:
        binding.svdmlp_destroy(h)
    _gpu.assert_close(Y, _gpu.oracle_rows(oracle, f, X, list(range(T))), f"T={T} r={r} ({path})")


@pytest.mark.parametrize("T", [2048, 1900])
def test_split_k_summed_inside_a_cluster(oracle, T):
    """Two K splits of the first projection on CTA pairs form one cluster and are summed through distributed shared
    memory (d = 1024 is 16 K chunks: exactly two splits at these T).  Against the oracle, every row, and against the
    same handle shape with the partial-buffer + reduction-launch form: both sum split 0 then split 1 in fp32, so the
    two forms give the same bits."""
    d, ffn, r = 1024, 2048, 256
    f = inputs.direct_factors(d, ffn, r, seed=8, device="cuda")
    X = inputs.activations(T, d, seed=8, device="cuda")
    Y = _gpu.run_mlp(f, X)
    Y_plain = _gpu.run_mlp(f, X, flags=binding.FLAG_NO_CLUSTER_SPLITK)
    _gpu.assert_close(Y, _gpu.oracle_rows(oracle, f, X, list(range(T))), f"cluster split-K T={T}")
    assert torch.equal(Y, Y_plain)


@pytest.mark.parametrize("T", [1, 8, 1024])
def test_cfg5_prenorm_residual_stack(oracle, T):
    d, ffn, r, L = 5120, 13824, 320, 40
    X = inputs.activations(T, d, seed=0, device="cuda")
    rows = inputs.sample_rows(T, max_rows=12)
    h_gpu = X.float()
    h_ref = oracle.to_f64(X[rows])
    worst_layer = 0.0
    for layer in range(L):
        f = inputs.direct_factors(d, ffn, r, seed=layer, device="cuda")
        hd = binding.svdmlp_create(*f.tensors(), max_T=T)
        h_next = binding.svdmlp_forward_prenorm_residual(hd, h_gpu, eps=1e-5)
        torch.cuda.synchronize()
        assert binding.svdmlp_last_device_status(hd) == 0
        binding.svdmlp_destroy(hd)
        if layer in (0, 17, 39):  # per-layer MLP output parity, from the GPU's own layer input
            hin = oracle.to_f64(h_gpu[rows])
            ref_delta = oracle.prenorm_residual(hin, [t.cpu() for t in f.tensors()]) - hin
            got_delta = (h_next[rows].double() - h_gpu[rows].double()).cpu().numpy()
            e = np.abs(got_delta - ref_delta).sum() / np.abs(ref_delta).sum()
            worst_layer = max(worst_layer, e)
        h_ref = oracle.prenorm_residual(h_ref, [t.cpu() for t in f.tensors()])
        h_gpu = h_next
    _gpu.assert_close(h_gpu[rows], h_ref, f"cfg5 T={T} final residual stream")
    delta_ref = h_ref - oracle.to_f64(X[rows])
    delta_gpu = (h_gpu[rows].double() - X[rows].double()).cpu().numpy()
    assert np.abs(delta_gpu - delta_ref).sum() / np.abs(delta_ref).sum() <= 1e-2
    assert worst_layer <= 1e-2  # the bf16 rounding of each layer's normalised input is inherent


@pytest.mark.parametrize("T", [33, 64, 129])
def test_cfg2_shapes_just_above_the_decode_limit(oracle, T):
    """The first token counts that leave the weight-streaming kernels (T > 32) and the first with two row tiles:
    full config-2 shapes, every row compared."""
    f = inputs.direct_factors(4096, 11008, 256, seed=0, device="cuda")
    X = inputs.activations(T, 4096, seed=3, device="cuda")
    h = binding.svdmlp_create(*f.tensors(), max_T=4096)  # a handle sized for prefill serves small T too
    assert binding.svdmlp_path_name(h, T) == "tensor"
    Y = binding.svdmlp_forward(h, X)
    torch.cuda.synchronize()
    assert binding.svdmlp_last_device_status(h) == 0
    binding.svdmlp_destroy(h)
    _gpu.assert_close(Y, oracle.svdmlp(X, *f.tensors()), f"cfg2 shapes T={T}")


def test_fp32_output_large_T_error_is_small(oracle):
    """fp32 Y on the tcgen05 path (TMEM-strip gate/up kernel): without the bf16 rounding of Y the error is that of
    the fp16 intermediates alone, far below the bf16-output figure."""
    T = 700
    f = inputs.direct_factors(4096, 11008, 256, seed=0, device="cuda")
    X = inputs.activations(T, 4096, seed=4, device="cuda")
    h = binding.svdmlp_create(*f.tensors(), max_T=T, flags=binding.FLAG_Y_FP32)
    Y = binding.svdmlp_forward(h, X)
    torch.cuda.synchronize()
    assert Y.dtype == torch.float32 and binding.svdmlp_last_device_status(h) == 0
    binding.svdmlp_destroy(h)
    rows = inputs.sample_rows(T, max_rows=32)
    mx, mean = _gpu.errors(Y[rows], _gpu.oracle_rows(oracle, f, X, rows))
    assert mx <= 2e-3 and mean <= 6e-4, (mx, mean)


def test_paths_agree_and_fp32_output(oracle):
    f = inputs.direct_factors(512, 1408, 64, seed=9, device="cuda")
    X = inputs.activations(200, 512, seed=9, device="cuda")
    ref = oracle.svdmlp(X, *f.tensors())
    Ys = _gpu.run_mlp(f, X, flags=SKINNY | binding.FLAG_Y_FP32)
    Yt = _gpu.run_mlp(f, X, flags=TENSOR | binding.FLAG_Y_FP32)
    assert Ys.dtype == torch.float32
    mx_s, mean_s = _gpu.assert_close(Ys, ref, "skinny fp32")
    mx_t, mean_t = _gpu.assert_close(Yt, ref, "tensor fp32")
    assert mean_s < 2e-4          # exact hi/lo intermediates: only fp32 accumulation error remains
    assert mean_t < 1e-3          # fp16 intermediates


@pytest.mark.parametrize("pairs", [0, binding.FLAG_NO_CTA_PAIRS])
def test_fp32_residual_ragged_tensor_path(oracle, pairs):
    # fp32 output + residual leave through [32 x 32] TMA stores: d not a multiple of 32, T not of 128
    d, ffn, r, T = 328, 1000, 72, 333
    f = inputs.direct_factors(d, ffn, r, seed=4, device="cuda")
    hin = inputs.activations(T, d, seed=4, device="cuda").float() * 3.0
    guard = torch.full((T + 2, d), 7.0, dtype=torch.float32, device="cuda")
    h = binding.svdmlp_create(*f.tensors(), max_T=T, flags=TENSOR | pairs)
    binding.svdmlp_forward_prenorm_residual(h, hin, eps=1e-5, h_out=guard[1:T + 1])
    torch.cuda.synchronize()
    assert binding.svdmlp_last_device_status(h) == 0
    binding.svdmlp_destroy(h)
    ref = oracle.prenorm_residual(oracle.to_f64(hin), [t.cpu() for t in f.tensors()])
    _gpu.assert_close(guard[1:T + 1], ref, "fp32 residual ragged")
    got_delta = (guard[1:T + 1].double() - hin.double()).cpu().numpy()
    ref_delta = ref - oracle.to_f64(hin)
    assert np.abs(got_delta - ref_delta).sum() / np.abs(ref_delta).sum() <= 1e-2
    assert torch.all(guard[0] == 7.0) and torch.all(guard[T + 1] == 7.0)


def test_decode_back_to_back_launches_many_ring_passes(oracle):
    # r = 1024 makes the persistent decode kernel walk its shared-memory ring several times per launch;
    # launches on two handles queue up without host synchronisation in between, as a serving loop does
    d, ffn, r, T = 4096, 14336, 1024, 8
    fs = [inputs.direct_factors(d, ffn, r, seed=s, device="cuda") for s in (0, 1)]
    hs = [binding.svdmlp_create(*f.tensors(), max_T=T) for f in fs]
    X = inputs.activations(T, d, seed=3, device="cuda")
    Ys = [torch.empty((T, d), dtype=torch.bfloat16, device="cuda") for _ in hs]
    for i in range(8):
        binding.svdmlp_forward(hs[i % 2], X, Ys[i % 2])
    torch.cuda.synchronize()
    for h, f, Y in zip(hs, fs, Ys):
        assert binding.svdmlp_last_device_status(h) == 0
        _gpu.assert_close(Y, oracle.svdmlp(X, *f.tensors()), "back-to-back decode")
        binding.svdmlp_destroy(h)


def test_bounded_wait_times_out_and_the_handle_stays_usable(oracle):
    # a wait that nothing satisfies gives up after its limit, reports SVDMLP_ERR_TIMEOUT and leaves the device usable
    f = inputs.direct_factors(256, 704, 32, seed=5, device="cuda")
    X = inputs.activations(8, 256, seed=5, device="cuda")
    h = binding.svdmlp_create(*f.tensors(), max_T=8)
    assert binding.svdmlp_last_device_status(h) == 0
    binding.svdmlp_selftest_timeout(h, limit_us=2000)
    assert binding.svdmlp_last_device_status(h) == -7          # SVDMLP_ERR_TIMEOUT, cleared by the read
    assert binding.svdmlp_last_device_status(h) == 0
    Y = binding.svdmlp_forward(h, X)
    torch.cuda.synchronize()
    assert binding.svdmlp_last_device_status(h) == 0
    _gpu.assert_close(Y, oracle.svdmlp(X, *f.tensors()), "forward after a timed-out wait")
    binding.svdmlp_destroy(h)


def test_zero_input_and_guard_bands():
    f = inputs.direct_factors(256, 704, 32, seed=1, device="cuda")
    for T, flags in ((8, 0), (300, 0)):
        buf = torch.full((T + 4, 256), 7.0, dtype=torch.bfloat16, device="cuda")
        X = torch.zeros((T, 256), dtype=torch.bfloat16, device="cuda")
        h = binding.svdmlp_create(*f.tensors(), max_T=T, flags=flags)
        binding.svdmlp_forward(h, X, buf[2:T + 2])
        torch.cuda.synchronize()
        assert torch.all(buf[2:T + 2] == 0)
        assert torch.all(buf[:2] == 7.0) and torch.all(buf[T + 2:] == 7.0)
        binding.svdmlp_destroy(h)


def test_repeated_calls_and_changing_T(oracle):
    f = inputs.direct_factors(256, 704, 32, seed=2, device="cuda")
    h = binding.svdmlp_create(*f.tensors(), max_T=300)
    for T in (8, 300, 3, 31, 129, 8):
        X = inputs.activations(T, 256, seed=T, device="cuda")
        Y = binding.svdmlp_forward(h, X)
        torch.cuda.synchronize()
        _gpu.assert_close(Y, oracle.svdmlp(X, *f.tensors()), f"repeat T={T}")
    assert binding.svdmlp_launch_count(h) >= 6
    with pytest.raises(binding.SvdMlpError):
        binding.svdmlp_forward(h, inputs.activations(301, 256, device="cuda"))
    binding.svdmlp_destroy(h)


def test_forward_host_matches_the_oracle(oracle):
    """The host-buffer entry point (the benchmark's end-to-end leg) against the oracle at the stated tolerances:
    default stream, then a side stream (the call records a graph and replays it: new contents in the same
    buffers), then a pageable output buffer (no direct stores into it)."""
    f = inputs.direct_factors(256, 704, 32, seed=2, device="cuda")
    fc = [t.cpu() for t in f.tensors()]
    for T in (8, 200):
        h = binding.svdmlp_create(*f.tensors(), max_T=T)
        X, X2 = inputs.activations(T, 256, seed=1), inputs.activations(T, 256, seed=5)
        ref, ref2 = oracle.svdmlp(X, *fc), oracle.svdmlp(X2, *fc)
        Xp, Yp = X.clone().pin_memory(), torch.empty((T, 256), dtype=torch.bfloat16).pin_memory()
        binding.svdmlp_forward_host(h, Xp, Yp)
        _gpu.assert_close(Yp, ref, f"host path T={T}, default stream")
        side = torch.cuda.Stream()
        for rep in range(3):
            Xp.copy_(X if rep == 0 else X2)
            Yp.zero_()
            binding.svdmlp_forward_host(h, Xp, Yp, stream=side)
            _gpu.assert_close(Yp, ref if rep == 0 else ref2, f"host path T={T}, side stream call {rep}")
        Ypage = torch.zeros((T, 256), dtype=torch.bfloat16)
        binding.svdmlp_forward_host(h, Xp, Ypage, stream=side)
        _gpu.assert_close(Ypage, ref2, f"host path T={T}, pageable output")
        assert binding.svdmlp_last_device_status(h) == 0
        binding.svdmlp_destroy(h)


@pytest.mark.parametrize("flags", [binding.FLAG_DECODE_REGISTERS, 0])
def test_partial_stage_mask_then_full_forward(oracle, flags):
    """The measurement hook that runs one kernel of the path leaves accumulators half-updated; once the mask is
    back to all stages the next full forward must be right again (small T: both decode kernel generations)."""
    f = inputs.direct_factors(264, 696, 40, seed=7, device="cuda")
    X = inputs.activations(8, 264, seed=7, device="cuda")
    h = binding.svdmlp_create(*f.tensors(), max_T=8, flags=flags)
    binding.svdmlp_stage_mask(h, 1)
    binding.svdmlp_forward(h, X)
    binding.svdmlp_stage_mask(h, 2)
    binding.svdmlp_forward(h, X)
    binding.svdmlp_stage_mask(h, 0xFFFFFFFF)
    Y = binding.svdmlp_forward(h, X)
    torch.cuda.synchronize()
    assert binding.svdmlp_last_device_status(h) == 0
    _gpu.assert_close(Y, oracle.svdmlp(X, *f.tensors()), "full forward after partial stage masks")
    binding.svdmlp_destroy(h)


def test_cooperative_launch_flag(oracle):
    f = inputs.direct_factors(1024, 2752, 64, seed=8, device="cuda")
    X = inputs.activations(8, 1024, seed=8, device="cuda")
    Y = _gpu.run_mlp(f, X, flags=binding.FLAG_DECODE_COOPERATIVE)
    _gpu.assert_close(Y, oracle.svdmlp(X, *f.tensors()), "cooperative decode launch")


@pytest.mark.parametrize("T,n_in,n_out,r", [(8, 256, 688, 32), (5, 264, 696, 40), (300, 264, 696, 40), (1024, 2048, 4096, 256),
                                            (100, 264, 696, 40), (1024, 8192, 16384, 4096),
                                            (512, 7168, 18432, 4096)])
def test_svdlinear_xuv_operator(oracle, T, n_in, n_out, r):
    # the last two cases are the shapes of the paper's standalone XUV kernel experiment (Section 5.2) at M = 1K and of
    # its block-size experiment (Section 5.3) at M = 512
    V = inputs.normal_tensor(11, 0, (r, n_in), scale=n_in ** -0.5, device="cuda")
    U = inputs.normal_tensor(11, 1, (n_out, r), scale=r ** -0.5, device="cuda")
    X = inputs.activations(T, n_in, seed=11, device="cuda")
    Y = binding.svdlinear_forward(X, U, V)
    torch.cuda.synchronize()
    rows = inputs.sample_rows(T, max_rows=32 if r <= 256 else 10)
    # bf16 output rounding alone costs ~1.4e-3 mean relative error
    _gpu.assert_close(Y[rows], oracle.svdlinear(X[rows], U, V), f"svdlinear T={T}")


def test_token_slab_schedule(oracle):
    """Gate/up and the first down product slab by slab over the tokens (three ragged slabs here: 5000 rows of
    ffn = 14336 are 143 MB of H): same result as the oracle, two rows of every 128-row tile compared."""
    T = 5000
    f = inputs.direct_factors(4096, 14336, 128, seed=0, device="cuda")
    X = inputs.activations(T, 4096, seed=2, device="cuda")
    Y = _gpu.run_mlp(f, X, flags=binding.FLAG_TOKEN_SLABS)
    rows = inputs.rows_of_every_tile(T, per_tile=2)
    _gpu.assert_close(Y[rows], _gpu.oracle_rows(oracle, f, X, rows), "token slabs")


@pytest.mark.parametrize("T,n_in,n_out,r", [(5, 264, 696, 40), (300, 264, 696, 40), (1024, 2048, 4096, 256)])
def test_svdlinear_handle(oracle, T, n_in, n_out, r):
    """svdlinear_create / svdlinear_apply: same operator, U re-encoded and maps built once; several T per handle."""
    V = inputs.normal_tensor(12, 0, (r, n_in), scale=n_in ** -0.5, device="cuda")
    U = inputs.normal_tensor(12, 1, (n_out, r), scale=r ** -0.5, device="cuda")
    h = binding.svdlinear_create(U, V, max_T=max(T, 64))
    for t in (T, min(T, 40), T):
        X = inputs.activations(t, n_in, seed=12 + t, device="cuda")
        Y = binding.svdlinear_apply(h, X)
        torch.cuda.synchronize()
        rows = inputs.sample_rows(t, max_rows=32)
        _gpu.assert_close(Y[rows], oracle.svdlinear(X[rows], U, V), f"svdlinear handle T={t}")
    with pytest.raises(binding.SvdMlpError):
        binding.svdlinear_apply(h, inputs.activations(max(T, 64) + 1, n_in, device="cuda"))
    binding.svdlinear_destroy(h)


@pytest.mark.parametrize("layout", [1, 2, 3])
@pytest.mark.parametrize("T,n_in,n_out,r", [(8, 264, 696, 40), (32, 264, 696, 40), (40, 264, 696, 40), (128, 264, 696, 40),
                                            (136, 264, 696, 40), (520, 264, 696, 40), (1024, 2048, 4096, 256)])
def test_svdlinear_transposed_layouts(oracle, T, n_in, n_out, r, layout):
    """Algorithm 2's is_XT / req_OT: X given as X^T[in, T] and / or Y wanted as Y^T[out, T].  Every element is compared
    (the oracle on X itself; a layout flag changes where elements sit, not their values), on shapes with ragged
    tiles in every dimension, on both sides of the 32-token and 128-token path boundaries."""
    V = inputs.normal_tensor(14, 0, (r, n_in), scale=n_in ** -0.5, device="cuda")
    U = inputs.normal_tensor(14, 1, (n_out, r), scale=r ** -0.5, device="cuda")
    X = inputs.activations(T, n_in, seed=14 + T, device="cuda")
    h = binding.svdlinear_create(U, V, max_T=T)
    try:
        Xin = X.t().contiguous() if layout & binding.X_TRANSPOSED else X
        out = binding.svdlinear_apply_layout(h, Xin, layout)
        plain = binding.svdlinear_apply(h, X)
        torch.cuda.synchronize()
    finally:
        binding.svdlinear_destroy(h)
    assert out.shape == ((n_out, T) if layout & binding.Y_TRANSPOSED else (T, n_out))
    Y = out.t() if layout & binding.Y_TRANSPOSED else out
    rows = list(range(T)) if T <= 520 else inputs.sample_rows(T, max_rows=48)
    _gpu.assert_close(Y[rows], oracle.svdlinear(X[rows], U, V), f"layout={layout} T={T}")
    if T > 32 and not layout & binding.X_TRANSPOSED:
        assert torch.equal(Y.contiguous(), plain)      # the same accumulators, stored elsewhere


def test_svdlinear_layout_argument_checks():
    V = inputs.normal_tensor(15, 0, (16, 64), scale=0.1, device="cuda")
    U = inputs.normal_tensor(15, 1, (64, 16), scale=0.1, device="cuda")
    h = binding.svdlinear_create(U, V, max_T=64)
    L = binding.lib()
    X = torch.zeros((64, 64), dtype=torch.bfloat16, device="cuda")
    Y = torch.zeros((64, 64), dtype=torch.bfloat16, device="cuda")
    assert L.svdlinear_apply_layout(h.ptr, X.data_ptr(), 12, Y.data_ptr(), 1, None) == -3     # T not a multiple of 8
    assert L.svdlinear_apply_layout(h.ptr, X.data_ptr(), 16, Y.data_ptr(), 4, None) == -1     # unknown flag
    assert L.svdlinear_apply_layout(h.ptr, X.data_ptr(), 12, Y.data_ptr(), 0, None) == 0
    torch.cuda.synchronize()
    binding.svdlinear_destroy(h)


def test_svdlinear_handle_reports_factors_outside_the_fp16_range():
    """A factor value beyond 65504 cannot be re-encoded for the large-T kernels: the handle says so (status -2) for
    T > 32 instead of returning inf/NaN, and still serves small T on the bf16 kernels."""
    V = inputs.normal_tensor(13, 0, (32, 256), scale=256 ** -0.5, device="cuda")
    U = inputs.normal_tensor(13, 1, (512, 32), scale=32 ** -0.5, device="cuda").clone()
    U[3, 5] = 1.0e5
    h = binding.svdlinear_create(U, V, max_T=128)
    X = inputs.activations(128, 256, seed=13, device="cuda")
    with pytest.raises(binding.SvdMlpError) as e:
        binding.svdlinear_apply(h, X)
    assert e.value.status == -2
    Y = binding.svdlinear_apply(h, X[:8].contiguous())
    torch.cuda.synchronize()
    assert torch.isfinite(Y.float()).all()
    binding.svdlinear_destroy(h)


@pytest.mark.parametrize("r,rd,T", [(72, 40, 1100), (64, 128, 1500), (128, 128, 1030), (32, 64, 2600)])
def test_fused_gateup_down1_ragged(oracle, r, rd, T):
    """Ranks up to 128: gate/up, SiLU and the first down product as one kernel with H kept in shared memory, on
    ragged shapes (partial last row strip, ffn tile and K chunk; one and two K chunks; several units per CTA pair),
    against the oracle and against the same handle shape with the fused kernel switched off."""
    d, ffn = 512, 2200
    f = inputs.direct_factors(d, ffn, r, seed=21, r_down=rd, device="cuda")
    X = inputs.activations(T, d, seed=21, device="cuda")
    rows = inputs.rows_of_every_tile(T, per_tile=3)
    ref = _gpu.oracle_rows(oracle, f, X, rows)
    Y = _gpu.run_mlp(f, X, flags=TENSOR)
    _gpu.assert_close(Y[rows], ref, f"fused r={r} rd={rd} T={T}")
    Y2 = _gpu.run_mlp(f, X, flags=TENSOR | binding.FLAG_NO_FUSED_DOWN1)
    _gpu.assert_close(Y2[rows], ref, f"unfused r={r} rd={rd} T={T}")


def test_fused_gateup_down1_repeated_launches(oracle):
    """Back-to-back forwards on one handle (ring phases, H buffers and the Zd accumulator carry over units, not launches)."""
    f = inputs.direct_factors(1024, 4096, 128, seed=22, device="cuda")
    h = binding.svdmlp_create(*f.tensors(), max_T=2048)
    for i, T in enumerate((2048, 1024, 2048)):
        X = inputs.activations(T, 1024, seed=30 + i, device="cuda")
        Y = binding.svdmlp_forward(h, X)
        torch.cuda.synchronize()
        assert binding.svdmlp_last_device_status(h) == 0
        rows = inputs.rows_of_every_tile(T, per_tile=2)
        _gpu.assert_close(Y[rows], _gpu.oracle_rows(oracle, f, X, rows), f"fused repeat {i}")
    binding.svdmlp_destroy(h)
