"""The C-ABI library loads, exports every function include/space.h declares, and
its host-only entry points agree with the oracle (no GPU needed)."""
import ctypes
import os
import re

import pytest

from oracle import layout as olayout

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def binding():
    from paper_2402_11809_b200 import build
    build.build()
    from paper_2402_11809_b200 import binding as b
    return b


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "space.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(space_[a-z_]+)\s*\(", text)))


def test_exports_match_header(binding):
    declared = _declared_functions()
    assert len(declared) >= 10 and "space_attn_step" in declared
    for name in declared:
        assert hasattr(binding.lib, name), name
    assert sorted(binding.EXPORTS) == declared


@pytest.mark.parametrize("k", range(1, 8))
@pytest.mark.parametrize("variant", [0, 1])
def test_space_layout_matches_oracle(binding, k, variant):
    lay = binding.space_layout(k, variant)
    name = olayout.SAME_GROUP if variant == 0 else olayout.EQ5_LITERAL
    n = olayout.n_block_rows(k)
    assert lay.k == k and lay.n_q == n
    assert [lay.mask[i] for i in range(n)] == olayout.block_mask_rows(k, name)
    assert [lay.relpos[i] for i in range(n)] == olayout.position_ids(k, 0, name)
    assert [lay.target_rows[t] for t in range(k + 1)] == olayout.target_rows(k)
    rows = olayout.block_rows(k)
    assert [(lay.group[i], lay.offset[i]) for i in range(n)] == rows
    assert [lay.kind[i] for i in range(n)] == [int(o != 0) for _, o in rows]


def test_host_side_errors(binding):
    lay = binding.Layout()
    assert binding.lib.space_layout(0, 0, ctypes.byref(lay)) == binding.E_INVALID_ARG
    assert binding.lib.space_layout(8, 0, ctypes.byref(lay)) == binding.E_INVALID_ARG
    assert binding.lib.space_layout(2, 5, ctypes.byref(lay)) == binding.E_INVALID_ARG
    assert binding.lib.space_layout(2, 0, None) == binding.E_INVALID_ARG
    for code in range(-6, 1):
        assert binding.space_strerror(code) != "unknown error"
    assert binding.space_strerror(-99) == "unknown error"
    good = dict(device=0, max_batch=4, n_q_heads=32, n_kv_heads=8, head_dim=128, k_max=5,
                vocab=32000, host_staging=0, s_cap=4096)
    assert binding.space_workspace_bytes(**good) > 0
    for bad in (dict(head_dim=96), dict(n_q_heads=24), dict(k_max=8), dict(max_batch=0), dict(s_cap=10)):
        assert binding.space_workspace_bytes(**{**good, **bad}) == 0
    h = ctypes.c_void_p()
    cfg = binding.Config(**{**good, "head_dim": 96})
    assert binding.lib.space_create(ctypes.byref(h), ctypes.byref(cfg)) == binding.E_UNSUPPORTED
    assert binding.lib.space_create(None, ctypes.byref(cfg)) == binding.E_INVALID_ARG
    assert binding.lib.space_attn_step(None, None, None) == binding.E_INVALID_ARG
    assert binding.lib.space_verify(None, None, None) == binding.E_INVALID_ARG
    assert binding.lib.space_kv_commit(None, None, None) == binding.E_INVALID_ARG


def test_create_without_device_reports_it(binding):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a CUDA device is present")
    with pytest.raises(binding.SpaceError) as e:
        binding.Context()
    assert e.value.code == binding.E_NO_DEVICE


def test_struct_sizes_match_c(binding):
    # compile a tiny C program against the header and compare sizeof()
    import subprocess, tempfile
    src = r'''
#include <stdio.h>
#include "space.h"
int main(void){ printf("%zu %zu %zu %zu %zu %zu %zu %zu %zu\n", sizeof(space_config), sizeof(space_layout_t),
  sizeof(space_attn_args), sizeof(space_verify_args), sizeof(space_commit_args), sizeof(space_host_step_args),
  sizeof(space_lmhead_args), sizeof(space_decode_state), sizeof(space_sar_args)); return 0; }
'''
    with tempfile.TemporaryDirectory() as d:
        open(os.path.join(d, "t.c"), "w").write(src)
        subprocess.check_call(["gcc", "-std=c99", "-I", os.path.join(ROOT, "include"),
                               os.path.join(d, "t.c"), "-o", os.path.join(d, "t")])
        out = subprocess.check_output([os.path.join(d, "t")]).decode().split()
    want = [ctypes.sizeof(x) for x in (binding.Config, binding.Layout, binding.AttnArgs,
                                       binding.VerifyArgs, binding.CommitArgs, binding.HostStepArgs,
                                       binding.LmHeadArgs, binding.DecodeState, binding.SarArgs)]
    assert [int(x) for x in out] == want
