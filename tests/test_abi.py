"""The C-ABI library loads and exports every symbol include/eesd.h declares; host-side
argument checking works without a GPU."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    from paper_2406_03853_b200 import build
    build.build()
    import paper_2406_03853_b200 as eesd
    return eesd.lib()


def test_every_declared_symbol_is_exported(L):
    hdr = open(os.path.join(ROOT, "include", "eesd.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    names = set(re.findall(r"\b(eesd_[a-z_]+)\s*\(", hdr))
    assert {"eesd_init", "eesd_prefill", "eesd_draft", "eesd_verify_accept", "eesd_generate"} <= names
    for n in names:
        assert hasattr(L, n), n


def test_header_is_plain_c(tmp_path):
    import shutil
    import subprocess
    src = tmp_path / "use_header.c"
    src.write_text('#include "eesd.h"\nint main(void) { eesd_config c; (void)c; return EESD_OK; }\n')
    gcc = shutil.which("gcc")
    if not gcc:
        pytest.skip("no C compiler")
    r = subprocess.run([gcc, "-std=c99", "-Wall", "-Wextra", "-Werror", "-I", os.path.join(ROOT, "include"), "-fsyntax-only", str(src)],
                       capture_output=True, text=True)
    assert r.returncode == 0, r.stderr


def test_layout_sizes_and_config_checks(L):
    from paper_2406_03853_b200 import binding as b
    import eesd_synth as synth
    from tests.helpers import config_from_spec
    for spec in (synth.TINY, synth.LLAMA2_13B, synth.LLAMA2_70B):
        cfg = config_from_spec(spec, max_ctx=1536)
        lay, sz = b.Layout(), b.Sizes()
        assert L.eesd_weight_layout(C.byref(cfg), C.byref(lay)) == 0
        assert L.eesd_required_bytes(C.byref(cfg), C.byref(sz)) == 0
        es = 4 if spec.dtype == "f32" else 2
        params = (spec.n_layers + 1) * spec.layer_params + (2 if spec.tie_exit_head else 3) * spec.vocab * spec.d_model
        assert params * es <= sz.weights_bytes <= params * es * 1.001 + (1 << 20)
        assert sz.kv_page_bytes == (spec.n_layers + 1) * 2 * spec.kv_dim * 16 * es
        assert sz.min_pages == 96
        assert (lay.exit_head == lay.lm_head) == spec.tie_exit_head
        assert lay.tiled == (0 if spec.dtype == "f32" else 1)      # bf16 models with tile-aligned shapes: tile-major matrices
        assert lay.cali_w == 0 and lay.cali_wp == 0
        cfg.controller, cfg.cali_sigma_m, cfg.cali_sigma_s = b.CTRL_CALI_TS, 0.2, 0.5
        lay2 = b.Layout()
        assert L.eesd_weight_layout(C.byref(cfg), C.byref(lay2)) == 0
        assert lay2.cali_w >= lay.total_bytes and lay2.total_bytes - lay.total_bytes >= (10 * spec.d_model ** 2) * es + 16 * spec.d_model
        cfg.cali_sigma_s = 0.0
        assert L.eesd_weight_layout(C.byref(cfg), C.byref(lay2)) == -1
    bad = config_from_spec(synth.TINY)
    bad.n_kv_heads = 3
    assert L.eesd_weight_layout(C.byref(bad), C.byref(lay)) == -1
    bad = config_from_spec(synth.TINY)
    bad.head_dim = 80
    assert L.eesd_required_bytes(C.byref(bad), C.byref(sz)) == -8
    bad = config_from_spec(synth.TINY, k_cap=16)
    assert L.eesd_required_bytes(C.byref(bad), C.byref(sz)) == -1
    assert L.eesd_strerror(-5).decode().startswith("context")
    assert L.eesd_prefill(None, None, 0) == -1 and L.eesd_generate(None, None, 0, 0, None, 0, None, None, None, None, 0, None) == -1


def test_tile_major_matrix_places_elements_where_the_header_says():
    import torch
    from paper_2406_03853_b200 import binding as b
    R, K = 256, 192
    flat = torch.zeros(2 * R * K)
    t = torch.arange(2 * R * K, dtype=torch.float32).view(2, R, K)
    m = b.TiledMatrix(flat, (2, R, K))
    m.copy_(t)
    for n, r, k in ((0, 0, 0), (0, 5, 70), (1, 129, 63), (1, 255, 191), (0, 128, 64)):
        pos = n * R * K + ((r // 128 * (K // 64) + k // 64) * 128 + r % 128) * 64 + k % 64
        assert flat[pos].item() == t[n, r, k].item()
    assert torch.equal(m.dense(), t)


def test_binding_refuses_to_run_without_cuda():
    import torch
    if torch.cuda.is_available():
        pytest.skip("CUDA present")
    import paper_2406_03853_b200 as eesd
    from tests.helpers import config_from_spec
    import eesd_synth as synth
    with pytest.raises(RuntimeError):
        eesd.Engine(config_from_spec(synth.TINY))


def test_attention_plan_never_needs_more_slices_than_can_be_merged(L):
    # every allowed page size, every context length up to what the configuration check admits, the
    # fewest and the most (head, row) pairs: at most 64 slices per head, slices of a whole number of
    # 16-position steps, every page covered, and a block never holds more than its kernel can
    from paper_2406_03853_b200 import binding as b
    for dtype, block_cap in ((b.F32, 192), (b.BF16, 256)):
        for pt in (8, 16, 32, 64, 128):
            limit = 12288
            pps, ns = C.c_int(), C.c_int()
            while L.eesd_attention_plan(dtype, limit, pt, 8, 1, 148, C.byref(pps), C.byref(ns)) != 0:
                limit -= pt
            assert limit >= 8192
            assert L.eesd_attention_plan(dtype, limit + 1, pt, 8, 1, 148, C.byref(pps), C.byref(ns)) == -8 or limit == 12288
            for ctx in list(range(1, 600)) + list(range(600, limit + 1, 97)) + [limit]:
                for hkv, pairs in ((1, 1), (8, 8), (40, 16), (8, 128), (1024, 1)):
                    pp, n = b.attention_plan(dtype, ctx, pt, hkv, pairs)
                    assert 1 <= n <= 64 and pp >= 1
                    assert (pp * pt) % 16 == 0
                    assert pp * pt <= max(block_cap, pt) + (8 if pt == 8 else 0)
                    assert pp * n >= (ctx + pt - 1) // pt > pp * (n - 1)
    # a configuration whose context could need more than 64 slices is refused
    from tests.helpers import config_from_spec
    import eesd_synth as synth
    cfg = config_from_spec(synth.TINY, max_ctx=8192 + 128, page_tokens=128)
    sz = b.Sizes()
    assert L.eesd_required_bytes(C.byref(cfg), C.byref(sz)) == -8
    cfg = config_from_spec(synth.TINY, max_ctx=8192, page_tokens=128)
    assert L.eesd_required_bytes(C.byref(cfg), C.byref(sz)) == 0
