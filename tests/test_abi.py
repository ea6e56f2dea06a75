"""The C-ABI library: it builds, loads without a GPU, exports every function the header declares,
and its host-side entry points behave (descriptor checks, record size, repacking)."""
import ctypes
import os
import re

import numpy as np
import pytest

from oracle import moe_oracle as orc
from workloads import synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2609_18063_b200 import build
    build.build()
    import paper_2609_18063_b200 as m
    return m


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "edg_moe.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"^\s*(?:int32_t|const char\*)\s+(\w+)\s*\(", text, flags=re.M)))


def test_library_exports_every_declared_symbol(lib):
    names = _declared_functions()
    assert {"prerouter_topk", "stage_experts_to_slots", "moe_expert_ffn_int4_lora", "moe_layer_decode"} <= set(names)
    raw = ctypes.CDLL(lib.LIB_PATH)
    for n in names:
        assert hasattr(raw, n), f"{n} is declared in edg_moe.h but not exported"
    assert set(lib.EXPORTS) == set(names), "binding and header disagree"
    assert lib.version() >= 1000


def test_record_bytes_and_desc_checks(lib):
    d2 = lib.make_desc(synth.CONFIGS["cfg2"])
    d1 = lib.make_desc(synth.CONFIGS["cfg1"])
    assert lib.record_bytes(d2) == orc.record_bytes(2048, 512, 64) == 1_769_472
    assert lib.record_bytes(d1) == orc.record_bytes(1024, 256, 32) == 491_520
    assert lib.check_desc(d2) == 0
    for field, bad in [("H", 2000), ("I", 96), ("group", 48), ("K", 33), ("E", 4), ("rank", 65),
                       ("n_adapters", 3), ("n_slots", 0), ("H", 8192)]:
        d = lib.make_desc(synth.CONFIGS["cfg2"])
        setattr(d, field, bad)
        assert lib.check_desc(d) == -2, field
    d = lib.make_desc(synth.CONFIGS["cfg2"]); d.out_dtype = 7
    assert lib.check_desc(d) == -1
    with pytest.raises(lib.EdgError):
        lib.record_bytes(d)
    assert lib.ffn_workspace_bytes(d2, 1) % 256 == 0
    assert lib.ffn_workspace_bytes(d2, 64) > lib.ffn_workspace_bytes(d2, 1)


def test_pack_unpack_identity_and_layout(lib):
    cfg = synth.CONFIGS["cfg1"]
    d = lib.make_desc(cfg)
    ex = synth.expert_tensors(cfg, 0, 5)
    rec = lib.pack_expert(d, ex)
    assert rec.nbytes == cfg.record_bytes
    back = lib.unpack_expert(d, rec)
    for proj in ("gate", "up", "down"):
        for a, b in zip(ex[proj], back[proj]):
            assert np.array_equal(np.asarray(a).view(np.uint8), np.asarray(b).view(np.uint8))
    # tile-major sections: chunk c (codes 32c..32c+31) of row n sits at ((n//16 * Kd/32 + c) * 16 + n%16) * 16,
    # with the canonical nibble order inside the chunk; (scale, zero) pairs at ((n//16 * Kd/g + gi) * 16 + n%16) * 4
    half = cfg.H * cfg.I // 2
    def code_off(Kd, n, c):
        return ((n // 16 * (Kd // 32) + c) * 16 + n % 16) * 16
    for n, c in [(0, 0), (5, 3), (17, 31), (255, 7)]:
        o = code_off(cfg.H, n, c)
        assert np.array_equal(rec[o:o + 16], ex["gate"][0][n, 16 * c:16 * c + 16])
        assert np.array_equal(rec[half + o:half + o + 16], ex["up"][0][n, 16 * c:16 * c + 16])
    n, gi = 21, 9
    o = 3 * half + ((n // 16 * (cfg.H // cfg.group) + gi) * 16 + n % 16) * 4
    sz = rec[o:o + 4].view(np.float16)
    assert sz[0] == ex["gate"][1][n, gi] and sz[1] == ex["gate"][2][n, gi]
    # down: four column slices of I/4 codes, each tile-major
    sw = cfg.I // 4
    n, c = 700, 5                                              # chunk 5 = codes 160..191 -> slice 2, chunk 1 of the slice
    o = 2 * half + (c // (sw // 32)) * (cfg.H * sw // 2) + code_off(sw, n, c % (sw // 32))
    assert np.array_equal(rec[o:o + 16], ex["down"][0][n, 16 * c:16 * c + 16])
    with pytest.raises(ValueError):
        lib.pack_expert(lib.make_desc(synth.CONFIGS["cfg2"]), ex)


def test_pack_accepts_exactly_the_zero_points_the_kernels_subtract_without_rounding(lib):
    """Zero points are fp16 values in [0, 16] that are multiples of 1/128: q - z then fits fp16's 11
    significant bits, whichever kernel forms it.  Anything else is refused and nothing is written."""
    cfg = synth.CONFIGS["cfg1"]
    d = lib.make_desc(cfg)
    ex = synth.expert_tensors(cfg, 0, 1)
    def with_zero(v, proj="up"):
        out = {p: tuple(np.array(a, copy=True) for a in t) for p, t in ex.items()}
        out[proj][2][3, 2] = np.float16(v)
        return out
    for ok in (0.0, 7.5, 3.25, 15.0, 16.0, 1.0 / 128, 9 + 5.0 / 128, 0.0078125 * 3):
        back = lib.unpack_expert(d, lib.pack_expert(d, with_zero(ok)))
        assert float(back["up"][2][3, 2]) == float(np.float16(ok))
    for bad, proj in ((0.1, "gate"), (17.0, "up"), (-1.0, "down"), (1.0 / 256, "up"), (4 + 1.0 / 256, "gate"),
                      (float("inf"), "down"), (float("nan"), "up")):
        rec = np.full(cfg.record_bytes, 0xA5, dtype=np.uint8)
        with pytest.raises(lib.EdgError) as ei:
            lib.pack_expert(d, with_zero(bad, proj), rec)
        assert ei.value.code == -4
        assert (rec == 0xA5).all()


def test_host_calls_reject_bad_handles(lib):
    import paper_2609_18063_b200.binding as b
    assert b._lib.edg_store_destroy(None) == -1
    assert b._lib.stage_experts_to_slots(None, 0, None, 0, None, None) == -1
    st = b.StoreStats()
    assert b._lib.edg_store_get_stats(None, ctypes.byref(st)) == -1
