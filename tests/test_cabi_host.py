"""Host-side checks that need no GPU: the library loads, exports what the header declares, and
rejects bad arguments before touching a device."""
import os
import re

import pytest

from paper_2510_25977_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    build.build()
    return binding.lib()


def test_every_declared_symbol_is_exported(L):
    header = "".join(open(os.path.join(ROOT, "include", n)).read() for n in ("svdmlp.h", "svdmlp_bench.h"))
    declared = set(re.findall(r"^(?:int|size_t|const char\*|unsigned long long)\s+(svd\w+)\s*\(", header, re.M))
    assert declared == set(binding.EXPORTS)
    for name in declared:
        assert hasattr(L, name), name


def test_flag_constants_match_the_header():
    header = open(os.path.join(ROOT, "include", "svdmlp.h")).read()
    flags = {m.group(1): int(m.group(2), 16) for m in re.finditer(r"#define SVDMLP_FLAG_(\w+)\s+(0x[0-9a-fA-F]+)u", header)}
    assert flags, "no flag definitions found"
    for name, value in flags.items():
        assert getattr(binding, "FLAG_" + name) == value, name
    assert len(set(flags.values())) == len(flags)  # no two flags share a bit pattern


def test_strerror_texts(L):
    assert binding.strerror(0) == "ok"
    texts = {binding.strerror(s) for s in range(-7, 1)}
    assert len(texts) == 8 and "unknown status" not in texts
    assert binding.strerror(-99) == "unknown status"


def test_create_rejects_bad_arguments_before_any_device_work(L):
    p = 0x1000  # fake, 16-byte aligned, never dereferenced on these paths
    good = dict(d=256, ffn=688, r_gate=32, r_up=32, r_down=32, Ug=p, Vg=p, Uu=p, Vu=p, Ud=p, Vd=p, max_T=16)
    def call(**kw):
        a = dict(good); a.update(kw)
        st, h = binding.svdmlp_create_raw(**a)
        assert not h.value
        return st
    assert call(d=0) == -1
    assert call(max_T=0) == -1
    assert call(Ug=0) == -1
    assert call(flags=binding.FLAG_PATH_SKINNY | binding.FLAG_PATH_TENSOR) == -1
    assert call(ffn=690) == -3
    assert call(r_down=12) == -3
    assert call(Vd=p + 8) == -3
    # valid arguments but no usable device here: must fail loudly (ARCH or CUDA), never succeed
    import torch
    if not torch.cuda.is_available():
        assert call() in (-4, -5)


def test_forward_and_linear_argument_checks(L):
    assert L.svdmlp_forward(None, 0x1000, 4, 0x1000, None) == -1
    assert L.svdmlp_destroy(None) == 0
    assert L.svdmlp_launch_count(None) == 0
    assert L.svdlinear_workspace_bytes(0, 8, 8, 8) == 0
    need = L.svdlinear_workspace_bytes(16, 256, 688, 32)
    assert need >= 16 * 32 * 4
    assert L.svdlinear_forward(0x1000, 16, 256, 688, 32, 0x1000, 0x1000, 0x1000, 0x1000, need, None) in (-4, -5, -3)
    assert L.svdlinear_forward(0x1000, 16, 256, 688, 32, 0x1000, 0x1000, 0x1000, 0x1100, need - 1, None) == -6
    assert L.svdlinear_forward(0x1000, 16, 250, 688, 32, 0x1000, 0x1000, 0x1000, 0x1100, need, None) == -3
    assert L.svdlinear_forward(0x1000, 0, 256, 688, 32, 0x1000, 0x1000, 0x1000, 0x1100, need, None) == -1


def test_block_aligned_rank_matches_eq5_and_the_oracle(oracle):
    # pure host arithmetic: safe without a GPU
    from paper_2510_25977_b200 import binding
    import itertools
    for (k, n), ratio, block in itertools.product([(4096, 11008), (4096, 14336), (5120, 13824), (2048, 8192), (256, 688)],
                                                   [0.0, 0.05, 0.1, 0.2, 0.5, 0.914, 0.99], [1, 16, 64, 128]):
        assert binding.svdmlp_block_aligned_rank(k, n, ratio, block) == oracle.block_aligned_rank(k, n, ratio, block)
    # closed form: at block 1 and alpha 0 the stored parameters r (k + n) never exceed (1 - ratio) k n
    for ratio in (0.05, 0.2, 0.8):
        r = binding.svdmlp_block_aligned_rank(4096, 11008, ratio, 1, 0.0)
        assert r * (4096 + 11008) <= (1 - ratio) * 4096 * 11008 < (r + 1) * (4096 + 11008)
    # the 0.05 ratio of the paper's end-to-end runs gives rank 2816 for a 4096 x 11008 projection
    assert binding.svdmlp_block_aligned_rank(4096, 11008, 0.05, 128) == 2816
    for bad in [(0, 8, 0.1, 16, 0.5), (8, 8, 1.0, 16, 0.5), (8, 8, -0.1, 16, 0.5), (8, 8, 0.1, 0, 0.5), (8, 8, 0.1, 16, 1.5)]:
        assert binding.lib().svdmlp_block_aligned_rank(*bad) == -1


def test_bench_reference_arm_prints_the_contract_line():
    """`bench.py --impl reference` times the oracle on the host cores and needs no GPU: one JSON line with the keys
    the measurement contract names."""
    import json
    import subprocess
    import sys
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1", "--warmup", "0"],
                         capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    j = json.loads(lines[0])
    assert j["impl"] == "reference" and j["metric"] == "svdmlp_fwd_tokens_per_s" and j["unit"] == "tokens/s"
    assert j["value"] > 0 and j["higher_is_better"] is True and j["vs_baseline"] is None
    assert j["config"]["workload"] == "cfg2_T8"
    assert j["cpu_baseline"]["kind"] == "oracle" and j["cpu_baseline"]["cores"] >= 1 and j["cpu_baseline"]["value"] == j["value"]
    assert j["e2e"] == {"value": j["value"], "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
