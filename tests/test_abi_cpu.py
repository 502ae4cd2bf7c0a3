"""Host-only checks of the C ABI: the library loads, exports every symbol that include/beagle.h
declares, and the entry points that need no GPU validate their arguments."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2505_24544_b200 import build
    from paper_2505_24544_b200.binding import load_library
    build.build()
    return load_library()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "beagle.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(beagle_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    from paper_2505_24544_b200.binding import EXPORTED_SYMBOLS
    names = declared_symbols()
    assert "beagle_prefill_kv" in names and "beagle_draft_step" in names
    assert "beagle_block_forward" in names and "beagle_verify_greedy" in names
    for n in names:
        assert hasattr(lib, n), f"{n} declared in beagle.h but not exported"
    assert sorted(EXPORTED_SYMBOLS) == names


def test_config_struct_matches_header():
    from paper_2505_24544_b200.binding import BeagleConfig, BeagleWeights
    assert C.sizeof(BeagleConfig) == 14 * 4                  # 12 int32 and 2 floats, no padding
    assert C.sizeof(BeagleWeights) == 13 * C.sizeof(C.c_void_p)      # eleven parameters + the optional FP8 LM head (codes, scales)


def good_config():
    from paper_2505_24544_b200.binding import BeagleConfig
    return BeagleConfig(4096, 32, 8, 128, 14336, 128256, 1, 1e-5, 1, 1, 32, 8192, 8)


def test_query_sizes_and_shape_validation(lib):
    from paper_2505_24544_b200.binding import BeagleConfig
    kv, ws = C.c_size_t(), C.c_size_t()
    cfg = good_config()
    assert lib.beagle_query_sizes(C.byref(cfg), C.byref(kv), C.byref(ws)) == 0
    assert kv.value == 2 * 32 * 8 * (8192 + 8) * 128 * 2
    assert ws.value > 0 and ws.value % 256 == 0
    assert lib.beagle_query_sizes(C.byref(cfg), None, C.byref(ws)) == 1
    bad = good_config(); bad.n_kv_heads = 5
    assert lib.beagle_query_sizes(C.byref(bad), C.byref(kv), C.byref(ws)) == 2
    bad = good_config(); bad.head_dim = 100
    assert lib.beagle_query_sizes(C.byref(bad), C.byref(kv), C.byref(ws)) == 2
    bad = good_config(); bad.head_dim = 256; bad.n_q_heads = 64; bad.n_kv_heads = 8       # bf16, 256-wide heads, 8 grouped heads: no kernel
    kv_, ws_ = C.c_size_t(), C.c_size_t()
    assert lib.beagle_query_sizes(C.byref(bad), C.byref(kv_), C.byref(ws_)) == 2
    ok = good_config(); ok.head_dim = 256; ok.n_q_heads = 32; ok.n_kv_heads = 8
    assert lib.beagle_query_sizes(C.byref(ok), C.byref(kv_), C.byref(ws_)) == 0
    bad = good_config(); bad.dtype = 7
    assert lib.beagle_query_sizes(C.byref(bad), C.byref(kv), C.byref(ws)) == 1
    # rotary option: a base below 1 (or negative) is rejected; a valid one adds the (cos, sin) table to the workspace
    bad = good_config(); bad.rope_theta = -1.0
    assert lib.beagle_query_sizes(C.byref(bad), C.byref(kv), C.byref(ws)) == 1
    rope = good_config(); rope.rope_theta = 500000.0
    ws2 = C.c_size_t()
    assert lib.beagle_query_sizes(C.byref(rope), C.byref(kv), C.byref(ws2)) == 0
    assert ws2.value - ws.value == (8192 + 8 + 1) * 64 * 8 + (-(8192 + 8 + 1) * 64 * 8) % 256
    bad = good_config(); bad.vocab = 0
    assert lib.beagle_query_sizes(C.byref(bad), C.byref(kv), C.byref(ws)) == 1
    n = C.c_size_t()
    assert lib.beagle_block_workspace_bytes(C.byref(cfg), 8, 2048, C.byref(n)) == 0 and n.value > 0
    assert lib.beagle_block_workspace_bytes(C.byref(cfg), 0, 2048, C.byref(n)) == 1
    # the training step's workspace contains the forward's
    g = C.c_size_t()
    assert lib.beagle_block_grad_workspace_bytes(C.byref(cfg), 8, 2048, C.byref(g)) == 0 and g.value > n.value and g.value % 256 == 0
    assert lib.beagle_block_grad_workspace_bytes(C.byref(cfg), 8, 0, C.byref(g)) == 1
    assert lib.beagle_block_grad_workspace_bytes(C.byref(cfg), 1 << 13, 1 << 13, C.byref(g)) == 3       # more than 2^24 positions


def test_packed_weights_bytes_counts_whole_tiles(lib):
    """Tile-major copies: every matrix padded to tiles of 128 rows x 128 bytes (64 bf16 / 128 FP8 elements)."""
    def tiles(n, k, elt):
        return -(-n // 128) * -(-(k * elt) // 128) * 128 * 128
    cfg = good_config()
    n = C.c_size_t()
    assert lib.beagle_packed_weights_bytes(C.byref(cfg), 0, C.byref(n)) == 0
    want = 2 * tiles(4096, 4096, 2) + 2 * tiles(1024, 4096, 2) + 2 * tiles(14336, 4096, 2) + tiles(4096, 14336, 2) + tiles(128256, 4096, 2)
    assert n.value == want
    assert lib.beagle_packed_weights_bytes(C.byref(cfg), 1, C.byref(n)) == 0
    assert n.value == want + tiles(128256, 4096, 1)
    odd = good_config(); odd.hidden = 520; odd.mlp_dim = 1416; odd.vocab = 4099; odd.n_q_heads = 8; odd.n_kv_heads = 2; odd.head_dim = 64
    assert lib.beagle_packed_weights_bytes(C.byref(odd), 0, C.byref(n)) == 0
    assert n.value == (tiles(512, 520, 2) + 2 * tiles(128, 520, 2) + tiles(520, 512, 2) + 2 * tiles(1416, 520, 2) + tiles(520, 1416, 2)
                       + tiles(4099, 520, 2))
    fp32 = good_config(); fp32.dtype = 0
    assert lib.beagle_packed_weights_bytes(C.byref(fp32), 0, C.byref(n)) == 0 and n.value == 0
    assert lib.beagle_packed_weights_bytes(C.byref(cfg), 0, None) == 1
    bad = good_config(); bad.n_kv_heads = 5
    assert lib.beagle_packed_weights_bytes(C.byref(bad), 0, C.byref(n)) == 2
    assert lib.beagle_pack_weights(None, None, 0, None) == 1


def test_null_context_is_rejected(lib):
    assert lib.beagle_prefill_kv(None, 0, None, None, None, None) == 1
    assert lib.beagle_draft_step(None, 0, None, None, 1, None, 1, None, None, None) == 1
    assert lib.beagle_verify_greedy(None, 0, 0, None, None, 0, None, None, None, None) == 1
    assert lib.beagle_block_forward(None, 1, 1, None, None, 1, 0, 1, None, None, None, None, 0, None) == 1
    assert lib.beagle_block_loss(None, 1, 1, None, None, 1, 0, 1, 0, None, 0, None, None, None, None, 0, None) == 1
    assert lib.beagle_block_grad(None, 1, 1, None, None, 1, 0, 1, 0, None, 0, None, 0.0, None, None, None, 0, None) == 1
    assert lib.beagle_verify_sample(None, 0, 0, None, None, None, 0, 1.0, None, None, None, None, None) == 1
    assert lib.beagle_draft_tree(None, 0, None, 1, 1, 1, None, None, None, None) == 1
    assert lib.beagle_quantize_rows_e4m3(None, 1, 4, 64, None, None, None) == 1
    assert lib.beagle_destroy(None) == 1
    assert lib.beagle_version().decode().startswith("beagle")


def test_create_rejects_bad_buffers(lib):
    from paper_2505_24544_b200.binding import BeagleWeights
    cfg = good_config()
    w = BeagleWeights()
    h = C.c_void_p()
    assert lib.beagle_create(C.byref(cfg), C.byref(w), 256, 1 << 40, 256, 1 << 40, C.byref(h)) == 1   # NULL weights
    for name, _ in BeagleWeights._fields_:
        setattr(w, name, 4096)
    assert lib.beagle_create(C.byref(cfg), C.byref(w), 256, 16, 256, 1 << 40, C.byref(h)) == 3        # cache too small
    assert lib.beagle_create(C.byref(cfg), C.byref(w), 257, 1 << 40, 256, 1 << 40, C.byref(h)) == 1   # misaligned
    assert not h.value
