"""CPU-side checks of the boundary: the library loads, exports every symbol the header declares,
and the host-only entry points (batch validation, status strings) behave.  No GPU needed."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from paper_2504_12397_b200 import binding as ab
from paper_2504_12397_b200 import workloads as wl
from paper_2504_12397_b200.build import build_library

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build_library()
    return ab.load_library()


def test_every_declared_symbol_is_exported(lib):
    text = open(os.path.join(ROOT, "include", "alora.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = set(re.findall(r"\b(alora_[a-z_]+)\s*\(", text))
    assert {"alora_create", "alora_register_adapter", "alora_prefill_layer", "alora_decode_step",
            "alora_full_lora_prefill_layer", "alora_project_qkv", "alora_kv_append", "alora_attend",
            "alora_forward_stack", "alora_batch_metadata", "alora_validate_batch"} <= names
    raw = C.CDLL(ab.LIB_PATH)
    for n in sorted(names):
        assert hasattr(raw, n), f"{n} declared in alora.h but not exported"


def test_status_strings(lib):
    seen = {ab.status_string(i) for i in range(10)}
    assert len(seen) == 10 and "ok" in seen
    assert ab.status_string(12345) == "unknown status"


def test_config_struct_matches_header():
    text = open(os.path.join(ROOT, "include", "alora.h")).read()
    body = text[text.index("typedef struct alora_config {"):text.index("} alora_config;")]
    fields = re.findall(r"^\s*(int32_t|float)\s+(\w+);", body, flags=re.M)
    assert [(("c_int" if t == "int32_t" else "c_float"), n) for t, n in fields] == \
        [(("c_int" if f[1] is C.c_int32 else "c_float"), f[0]) for f in ab.alora_config._fields_]


def test_create_without_device_fails_loudly(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    cfg = ab.make_config(hidden=256, n_q_heads=4, n_kv_heads=2, head_dim=64, max_tokens=16, max_requests=1)
    with pytest.raises(ab.AloraError) as e:
        ab.alora_create(cfg)
    assert e.value.status == 9  # ALORA_ERR_NO_DEVICE


def _cfg(**kw):
    base = dict(hidden=256, n_q_heads=4, n_kv_heads=2, head_dim=64, page_size=4, max_tokens=64, max_requests=8,
                max_adapters=2)
    base.update(kw)
    return ab.make_config(**base)


def _batch():
    shape = wl.LayerShape(256, 4, 2, 64, page_size=4, dtype="fp32")
    return wl.make_batch(shape, [7, 12, 0], [5, 3, 9], [0, 1, -1], np.random.default_rng(0), shuffle_pages=True,
                         with_hidden=False)


def _validate(cfg, b, **over):
    a = dict(positions=b.positions, activation_offsets=b.activation_offsets, adapter_ids=b.adapter_ids,
             query_start_loc=b.query_start_loc, seq_lens=b.seq_lens, block_tables=b.block_tables,
             num_pages=b.num_pages)
    a.update(over)
    return ab.alora_validate_batch(cfg, **a)


def test_validate_batch_accepts_good_and_rejects_bad(lib):
    cfg, b = _cfg(), _batch()
    assert _validate(cfg, b) == 0
    pos = b.positions.copy(); pos[2] += 1
    assert _validate(cfg, b, positions=pos) == 6                       # positions not consecutive
    sl = b.seq_lens.copy(); sl[0] += 1
    assert _validate(cfg, b, seq_lens=sl) == 6                         # positions do not end at seq_len - 1
    ids = b.adapter_ids.copy(); ids[0] = 2
    assert _validate(cfg, b, adapter_ids=ids) == 6                     # adapter id beyond max_adapters
    bt = b.block_tables.copy(); bt[1, 0] = b.num_pages
    assert _validate(cfg, b, block_tables=bt) == 7                     # page id outside the pool
    bt = b.block_tables.copy(); bt[1, 3] = bt[0, 2]
    assert _validate(cfg, b, block_tables=bt) == 6                     # two requests would write one page
    q = b.query_start_loc.copy(); q[-1] += 1
    assert _validate(cfg, b, query_start_loc=q) == 6
    assert _validate(_cfg(max_tokens=8), b) == 3                       # capacity
    a = b.activation_offsets.copy(); a[0] = -1
    assert _validate(cfg, b, activation_offsets=a) == 6


def test_validate_batch_allows_shared_read_only_prefix_pages(lib):
    """Two requests may point at the same physical prefix pages as long as neither writes them."""
    cfg = _cfg()
    shape = wl.LayerShape(256, 4, 2, 64, page_size=4, dtype="fp32")
    b = wl.make_batch(shape, [8, 8], [3, 3], [0, 1], np.random.default_rng(1), with_hidden=False)
    bt = b.block_tables.copy()
    bt[1, :2] = bt[0, :2]  # both prefixes (2 full pages) are the same physical pages
    assert _validate(cfg, b, block_tables=bt) == 0


def test_missing_library_is_reported(tmp_path, monkeypatch):
    monkeypatch.setattr(ab, "_lib", None)
    monkeypatch.setattr(ab, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(ab.AloraLibraryMissing):
        ab.load_library()


def test_projection_item_order_never_waits_for_a_block_that_is_not_running():
    """Host-side model of the order in which a projection launch's blocks take their items (csrc/claim_order.h, the
    two decisions the kernels use): with shrink items claimed from a counter every item completes however few blocks
    are running and whichever blocks start first; dealing all items by block index (the order it replaced) leaves
    running blocks waiting for shrink items of blocks that never get a slot."""
    from paper_2504_12397_b200 import binding as ab
    for grid, n_shrink, rows, cols in ((148, 16, 16, 24), (148, 200, 264, 24), (8, 3, 5, 2), (4, 9, 9, 1), (148, 1, 40, 32)):
        for slots in (1, 2, 7, grid):
            for high_first in (True, False):
                assert ab.alora_selftest_claim_order(grid, n_shrink, rows, cols, slots, high_first), (grid, n_shrink, slots, high_first)
    # the replaced order: fine when every block runs, stuck when the low blocks cannot start
    assert ab.alora_selftest_claim_order(148, 16, 16, 24, 148, True, static_order=True)
    assert not ab.alora_selftest_claim_order(148, 16, 16, 24, 100, True, static_order=True)
    assert not ab.alora_selftest_claim_order(8, 3, 5, 2, 2, True, static_order=True)
    # no shrink items at all (a base-only launch): nothing to claim, nothing to wait for
    assert ab.alora_selftest_claim_order(148, 0, 16, 24, 3, True)
