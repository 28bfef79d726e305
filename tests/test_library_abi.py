"""The C-ABI library builds, loads without a GPU and exports every function include/seer.h declares; the host-only
sizing helpers compute the closed forms of the layout."""
import os
import re

import pytest

from paper_2410_13276_b200 import binding as B, build as build_mod


@pytest.fixture(scope="module")
def lib():
    build_mod.build()
    return B.load_library()


def declared_functions(repo_root):
    text = open(os.path.join(repo_root, "include", "seer.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(seer_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported_and_bound(lib, repo_root):
    names = declared_functions(repo_root)
    assert "seer_gate_scores" in names and "seer_block_mask" in names and "seer_sparse_attn" in names
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in seer.h but not exported"
    assert sorted(B.EXPORTS) == names, "binding.EXPORTS and seer.h disagree"


def test_sizing_helpers_closed_forms(lib):
    s = B.make_shape([0, 131072], 32, 8)
    assert B.seer_mask_rows(s) == 32 * 2048
    assert B.seer_scores_elems(s) == 32 * 2048 * 2048
    assert B.seer_causal_blocks(s) == 32 * 2048 * 2049 // 2 == 67141632
    assert B.seer_workspace_bytes(s) == (32 + 8) * 2048 * 128 * 6     # projected pooled Q, K: three bf16 planes each
    v = B.make_shape([0, 8192, 8192 + 16384, 8192 + 16384 + 32768, 122880], 40, 8)
    assert B.seer_mask_rows(v) == 40 * (128 + 256 + 512 + 1024) == 76800
    assert B.seer_causal_blocks(v) == 27891200
    r = B.make_shape([0, 65, 65, 130], 2, 1)                 # ragged, with an empty sequence
    assert B.seer_mask_rows(r) == 2 * (2 + 0 + 2) and B.seer_scores_elems(r) == 2 * (4 + 0 + 4)
    # 128-token gate blocks: a quarter of the score matrix, half the rows; other block sizes are rejected
    s128 = B.make_shape([0, 131072], 32, 8, block=128)
    assert B.seer_mask_rows(s128) == 32 * 1024 and B.seer_scores_elems(s128) == 32 * 1024 * 1024
    assert B.seer_causal_blocks(s128) == 32 * 1024 * 1025 // 2
    r128 = B.make_shape([0, 65, 65, 194], 2, 1, block=128)   # 65 tokens: one block of 128, two of 64
    assert B.seer_mask_rows(r128) == 2 * (1 + 0 + 2)
    assert B.seer_mask_rows(B.make_shape([0, 128], 2, 1, block=32)) == -1
    assert B.seer_mask_rows(B.make_shape([0, 128], 2, 1, block=256)) == -1
    # gate + mask in one call: the projected vectors plus the band scratch, never less than 64 rows of the longest sequence
    assert B.seer_gate_mask_workspace_bytes(s, 128 << 20) == B.seer_workspace_bytes(s) + (128 << 20)
    assert B.seer_gate_mask_workspace_bytes(s, 0) == B.seer_workspace_bytes(s) + (64 * 2048 + 4) * 4 + 240
    # the host-buffer path works on one KV head (4 query heads) at a time: two sets of slice inputs / outputs
    # (q, o: 2 x 2 x 134 MB; k, v: 2 x 2 x 33.5 MB) and one set of slice intermediates (scores 67 MB, lists 33.6 MB)
    assert 0.75e9 < B.seer_prefill_host_arena_bytes(s) < 0.85e9


def test_invalid_shapes_are_rejected_without_a_gpu(lib):
    assert B.seer_mask_rows(B.make_shape([0, 128], 3, 2)) == -1          # Hq not a multiple of Hkv
    assert B.seer_mask_rows(B.make_shape([0, 128], 2, 1, head_dim=64)) == -1
    assert B.seer_mask_rows(B.make_shape([0, 128, 64], 2, 1)) == -1      # decreasing offsets
    assert B.seer_workspace_bytes(B.make_shape([5, 128], 2, 1)) == 0     # cu[0] != 0
    assert B.seer_status_string(4) == "col_idx capacity exceeded"


def test_context_creation_fails_loudly_without_a_device(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    with pytest.raises(B.SeerError) as e:
        B.Context(0)
    assert e.value.status == 7
