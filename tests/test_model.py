"""The capacity / intensity model (svdmlp_model: the role Eq. 10 and Eq. 11 play in Section 4.2.1 "Blocking",
restated for an sm_100 SM).  Host arithmetic only, so these run without a GPU."""
import pytest

from paper_2510_25977_b200 import binding, build


@pytest.fixture(scope="module", autouse=True)
def _lib():
    build.build()
    binding.lib()


def test_flops_and_hbm_bytes_are_the_counts_of_the_paper():
    d, ffn, r, T = 4096, 11008, 256, 8
    m = binding.svdmlp_model(d, ffn, r, T)
    assert m["flops"] == 2 * T * r * (3 * d + 3 * ffn)              # Section 3: 2 T r (k + n) per projection
    assert m["hbm_bytes"] == 2 * (3 * r * (d + ffn)) + 2 * 2 * T * d  # factors once, X in, Y out (16-bit)
    assert m["t_hbm_us"] == pytest.approx(m["hbm_bytes"] / 6547e3)
    assert m["t_floor_us"] == max(m["t_hbm_us"], m["t_tensor_us"])
    assert m["ridge_hbm"] == pytest.approx(1648e3 / 6547)


def test_intensity_follows_eq10_in_the_strip_height(oracle):
    """Eq. 10: per row strip of B_M rows the factors are read once more.  The model's bytes between two batch sizes
    that differ by one whole strip grow by one pass over the factors plus that strip's activations; and for one
    projection alone (activations of the other two removed) the intensity is Eq. 10's."""
    d, ffn, r = 5120, 14336, 512
    a, b = binding.svdmlp_model(d, ffn, r, 512), binding.svdmlp_model(d, ffn, r, 768)
    assert a["strip_rows"] == b["strip_rows"] == 256
    factors = 2 * 3 * r * (d + ffn)
    acts = 256 * 2 * (2 * d + 2 * 3 * r + 2 * ffn)                    # X, Y; Z and Zd out and back; H out and back
    assert b["sm_bytes"] - a["sm_bytes"] == factors + acts
    # the factor term alone, against Eq. 10 with K + N = d + ffn: 2 M r (K+N) / (s (M/B_M) r (K+N)) = 2 B_M / s ... plus the
    # activation term M (K+N): together Eq. 10
    M, B_M, s = 768, 256, 2
    eq10 = oracle.arithmetic_intensity(r, B_M, s)
    one_projection = 2 * M * r * (d + ffn) / (s * (M * (d + ffn) + (M // B_M) * r * (d + ffn)))
    assert one_projection == pytest.approx(eq10)
    three_separate = 3 * s * (M * (d + ffn) + (M // B_M) * r * (d + ffn))
    assert b["sm_bytes"] < three_separate                              # fusion: X read once, G and Up never leave the SM
    assert b["intensity_sm"] > eq10 * 0.99


def test_intensity_grows_with_the_batch_and_saturates():
    d, ffn, r = 4096, 11008, 256
    vals = [binding.svdmlp_model(d, ffn, r, T)["intensity_sm"] for T in (64, 128, 256, 2048, 8192)]
    assert vals[0] < vals[1] < vals[2]            # below one strip every token adds flops, not factor bytes
    assert vals[3] == pytest.approx(vals[4], rel=0.02)   # whole strips: flat, Eq. 10 with B_M fixed


@pytest.mark.parametrize("d,ffn,r,T,path,z_in_tmem", [
    (4096, 11008, 256, 8, 0, 0), (4096, 11008, 256, 32, 0, 0), (5120, 14336, 1024, 16, 0, 0),
    (5120, 14336, 1024, 32, 1, 0),        # the decode kernel's Z rows do not fit next to its ring
    (4096, 11008, 256, 4096, 1, 1),       # Z strip as TMEM-resident A operand
    (5120, 14336, 512, 2048, 1, 0),       # strip too wide for TMEM: both operands streamed
    (5120, 14336, 128, 2048, 2, 1), (5120, 14336, 128, 128, 2, 1), (256, 688, 32, 64, 1, 0)])   # too few ffn tiles to fill the SM pairs: not fused
def test_paths_and_on_chip_budgets(d, ffn, r, T, path, z_in_tmem):
    m = binding.svdmlp_model(d, ffn, r, T)
    assert (m["path"], m["z_in_tmem"]) == (path, z_in_tmem)
    assert m["tmem_cols_total"] == m["tmem_cols_strip"] + m["tmem_cols_acc"] + m["tmem_cols_zd"] <= 512   # Eq. 11's role
    assert 0 < m["smem_bytes"] <= 232448
    if path == 2:
        assert m["tmem_cols_zd"] >= r and m["tmem_cols_strip"] >= r       # packed fp16 gate + up strip: r columns
    if path == 0:
        assert m["tmem_cols_total"] == 0 and m["strip_rows"] in (8, 16, 32)


def test_h_round_trip_counts_only_beyond_l2():
    d, ffn, r = 5120, 14336, 512
    small, big = binding.svdmlp_model(d, ffn, r, 2048), binding.svdmlp_model(d, ffn, r, 8192)
    base = lambda T: 2 * 3 * r * (d + ffn) + 4 * T * d
    assert small["hbm_bytes"] == base(2048)                               # H = 59 MB stays in the 126 MB L2
    assert big["hbm_bytes"] == base(8192) + 2 * 2 * 8192 * ffn            # H = 235 MB: written and read through HBM
    assert binding.svdmlp_model(d, ffn, 128, 8192)["hbm_bytes"] == 2 * 3 * 128 * (d + ffn) + 4 * 8192 * d   # fused: no H


def test_argument_checks():
    with pytest.raises(binding.SvdMlpError):
        binding.svdmlp_model(0, 11008, 256, 8)
    assert binding.lib().svdmlp_model(4096, 11008, 256, 8, 0.0, 0.0, 0.0, None) == -1
