"""The C-ABI library builds, loads without a GPU and exports every symbol the header declares."""
import ctypes
import os
import re

from paper_2509_15038_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "curdkv.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(curdkv_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib_path = build.build_library()
    lib = ctypes.CDLL(str(lib_path))
    names = declared_functions()
    assert len(names) >= 7
    for name in names:
        assert hasattr(lib, name), f"{name} is declared in curdkv.h but not exported"
    assert set(binding.EXPORTS) == set(names)


def test_host_only_calls_work_without_a_device():
    lib = binding.load()
    assert binding.status_string(0) == "ok"
    assert "workspace" in binding.status_string(3)
    desc = binding.Desc(4, 8, 32, 1000, 128, 32, 0, 0, 128, 0, 0, 128, None, 0, 1)
    # 256 status bytes + four fp32 partials per 128-row tile, rounded to 256 bytes
    assert binding.workspace_bytes(desc) == 256 + 4 * 8 * 8 * 4 * 4
    bad = binding.Desc(4, 8, 12, 1000, 128, 32, 0, 0, 128, 0, 0, 128, None, 0, 1)
    assert binding.workspace_bytes(bad) == 0
    assert lib.curdkv_score(None, None, None, 0, None, None, None, None, 0, None) == 1


def test_workspace_sizes_of_the_added_modes_without_a_device():
    lib = binding.load()
    plain = binding.Desc(4, 8, 32, 1000, 128, 32, 0, 0, 128, 0, 0, 128, None, 0, 1)
    white = binding.Desc(4, 8, 32, 1000, 128, 32, 0, 0, 128, 0, 0, 128, None, 0, 1, 0, 1, 1e-4)
    base = binding.workspace_bytes(plain)
    # whitened: + one partial Gram pair (2 x 128 x 128 fp32) per (head, segment) + W (2 x 128 x r fp32) per head
    extra = binding.workspace_bytes(white) - base
    heads = 4 * 8
    assert extra >= heads * 2 * 128 * 128 * 4 + heads * 2 * 128 * 32 * 4
    assert extra % (2 * 128 * 128 * 4) % 256 == 0
    bad_ridge = binding.Desc(4, 8, 32, 1000, 128, 32, 0, 0, 128, 0, 0, 128, None, 0, 1, 0, 1, -1.0)
    assert binding.workspace_bytes(bad_ridge) == 0
    # generation-phase cache: grows with rows appended per call and with the budget
    small = lib.curdkv_cache_workspace_bytes(4, 8, 16, 512, 256)
    assert small > 0
    assert lib.curdkv_cache_workspace_bytes(4, 8, 256, 512, 256) > small
    assert lib.curdkv_cache_workspace_bytes(4, 8, 16, 512, 400) > small
    assert lib.curdkv_cache_workspace_bytes(4, 0, 16, 512, 256) == 0
    # evaluator: status words + one int32 per head
    import ctypes as ct
    assert lib.curdkv_attention_workspace_bytes(ct.byref(plain)) == 256 + 256
    # calls with NULL arguments are refused on the host, nothing is launched
    before = binding.launch_count()
    assert lib.curdkv_cache_compress(None, None, None, 1, 0, 0, None, 0, None) == 1
    assert lib.curdkv_eviction_loss(None, None, 1, 1, None, None, None) == 1
    assert lib.curdkv_gqa_expand(None, None, None, 1, None, None, None) == 1
    assert binding.launch_count() == before


def _whiten_segments(batch, heads, n, r=32):
    """Segments per head the library plans for a whitened call, read off its workspace size."""
    plain = binding.Desc(batch, heads, heads, n, 128, r, 0, 0, 128, 0, 0, 128, None, 0, 1)
    white = binding.Desc(batch, heads, heads, n, 128, r, 0, 0, 128, 0, 0, 128, None, 0, 1, 0, 1, 1e-4)
    extra = binding.workspace_bytes(white) - binding.workspace_bytes(plain)
    P = batch * heads
    w_bytes = -(-(P * 2 * 128 * r * 4) // 256) * 256
    return (extra - w_bytes) // (P * 2 * 128 * 128 * 4)


def test_whitened_segment_count_follows_the_cost_model():
    """Segments per head minimise ceil(P s / SMs) x (tiles per item + 10) over s (host logic only;
    without a device the library plans for a B200's 148 SMs, which is also what a B200 reports):
    the three bench shapes, and a single long head, which must be cut up to feed all SMs."""
    sms = 148

    def model(P, tiles):
        cost = lambda s: -(-(P * s) // sms) * (-(-tiles // s) + 10)
        return min(range(1, min(tiles, 1024) + 1), key=lambda s: (cost(s), s))
    for batch, heads, n in [(32, 8, 8192), (128, 8, 32768), (32, 8, 131072), (1, 1, 131072), (1, 2, 1000)]:
        tiles = -(-n // 128)
        assert _whiten_segments(batch, heads, n) == model(batch * heads, tiles), (batch, heads, n)
    assert _whiten_segments(32, 8, 8192) == 1 and _whiten_segments(32, 8, 131072) == 4
    assert _whiten_segments(1, 1, 131072) == 147          # 147 items of 7 tiles: one round on 148 SMs
