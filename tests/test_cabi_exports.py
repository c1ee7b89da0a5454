"""CPU-only checks of the boundary: the library loads without a GPU, exports every function the
header declares, and rejects bad configurations on the host before touching CUDA."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "saem.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(saem_[a-z_]+)\s*\(", text)))


def test_library_loads_and_exports_every_declared_symbol():
    from paper_2608_21614_b200 import binding as B
    lib = ctypes.CDLL(B.library_path())
    names = _declared()
    assert len(names) >= 20
    for n in names:
        assert hasattr(lib, n), "missing export " + n
    assert sorted(B.EXPORTS) == names
    for n in names:
        assert hasattr(B, n), "binding lacks " + n


def test_host_side_validation_needs_no_gpu():
    from paper_2608_21614_b200 import binding as B
    good = B.make_config(512, 1024, 8, 2, 64)
    assert B.saem_slot_bytes(good) == 3 * 512 * 1024 * 2
    assert B.saem_slot_region_bytes(good) == 8 * B.saem_slot_bytes(good)
    assert B.saem_workspace_bytes(good) > 64 * 2 * 1024 * 2
    for bad in (B.make_config(500, 1024, 8, 2, 64), B.make_config(512, 1000, 8, 2, 64),
                B.make_config(512, 1024, 129, 2, 64), B.make_config(512, 1024, 8, 9, 64),
                B.make_config(512, 1024, 8, 2, 0), B.make_config(512, 1024, 8, 2, 40000)):
        assert B.saem_slot_bytes(bad) == 0 and B.saem_workspace_bytes(bad) == 0
        assert B.saem_create_status(bad, 1024, 1 << 40, 2048, 1 << 40) == B.SAEM_ERR_SHAPE
    assert B.saem_create_status(good, 0, 1 << 40, 2048, 1 << 40) == B.SAEM_ERR_INVALID_ARG
    assert B.saem_create_status(good, 1024 + 8, 1 << 40, 2048, 1 << 40) == B.SAEM_ERR_ALIGNMENT
    assert B.saem_create_status(good, 1024, 100, 2048, 1 << 40) == B.SAEM_ERR_WORKSPACE
    assert B.saem_create_status(good, 1024, 1 << 40, 2048, 100) == B.SAEM_ERR_WORKSPACE
    assert B.saem_status_string(B.SAEM_ERR_TIMEOUT)


def test_weight_packer_is_a_permutation_of_the_input_bytes():
    """Host-only: the slot layout holds exactly the expert's values, each once (tile + swizzle)."""
    import numpy as np
    from paper_2608_21614_b200 import binding as B
    d, f = 128, 256
    cfg = B.make_config(d, f, 1, 1, 4)
    n = d * f
    gate = np.arange(0, n, dtype=np.uint32).astype(np.uint16).reshape(f, d)
    up = (np.arange(0, n, dtype=np.uint32) + n).astype(np.uint16).reshape(f, d)
    down = (np.arange(0, n, dtype=np.uint32) + 2 * n).astype(np.uint16).reshape(d, f)   # 3n = 98304 > 65535 wraps
    out = np.zeros(B.saem_slot_bytes(cfg) // 2, np.uint16)
    B.saem_pack_expert_host(cfg, gate, up, down, out)
    assert np.array_equal(np.sort(out), np.sort(np.concatenate([gate.ravel(), up.ravel(), down.ravel()])))
    # first gate tile, row r, 16-byte chunk c sits at chunk c ^ (r & 7)
    tile = out[:128 * 64].reshape(128, 8, 8)
    for r in (0, 1, 7, 9, 127):
        for c in (0, 3, 7):
            assert np.array_equal(tile[r, c ^ (r & 7)], gate[r, c * 8:(c + 1) * 8])
    # the matching up tile follows the gate tile
    tile_u = out[128 * 64:2 * 128 * 64].reshape(128, 8, 8)
    assert np.array_equal(tile_u[5, 2 ^ 5], up[5, 16:24])


def test_header_constants_match_the_binding_and_large_repack_shapes_are_accepted():
    """The enumerators of include/saem.h have the values the ctypes binding uses, and the shapes that the
    one-CTA repack index phase used to refuse (128 experts top-8 beyond 2560 tokens) are valid configs."""
    from paper_2608_21614_b200 import binding as B
    text = open(os.path.join(ROOT, "include", "saem.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    consts = dict((k, int(v)) for k, v in re.findall(r"\b(SAEM_[A-Z0-9_]+)\s*=\s*(-?\d+)\s*[,}]", text))
    consts["SAEM_STATIC_SCRATCH_ELEMS"] = 1 << 20                                  # written as 1 << 20 in the header
    assert re.search(r"SAEM_STATIC_SCRATCH_ELEMS\s*=\s*1\s*<<\s*20", text)
    assert len(consts) >= 20
    for name, value in consts.items():
        assert getattr(B, name) == value, name
    for E, k, T in ((128, 8, 4096), (64, 5, 13107), (9, 1, 40000)):
        cfg = B.make_config(128, 128, E, k, T)
        assert B.saem_slot_bytes(cfg) > 0 and B.saem_workspace_bytes(cfg) > 0
    assert B.saem_slot_bytes(B.make_config(128, 128, 64, 5, 13108)) == 0          # 65 540 pairs: one too many tokens
    assert B.make_config(128, 128, 8, 2, 4, ffn_path=B.SAEM_FFN_DECODE_FUSED).ffn_path == 4
