"""The C-ABI library builds for sm_100a, loads without a GPU and exports every
symbol include/less.h declares; host-side argument checks answer with error
codes (no compute calls here)."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def B():
    from paper_2402_09398_b200 import build, binding
    build.build()
    binding.lib()
    return binding


def declared_functions():
    text = open(os.path.join(ROOT, "include", "less.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(less_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(B):
    names = declared_functions()
    assert "less_create" in names and "less_decode_step" in names and "less_prefill" in names
    L = B.lib()
    for n in names:
        assert hasattr(L, n), f"{n} declared in less.h but not exported"
    assert sorted(B.EXPORTED) == names


def test_config_validation(B):
    def cfg(**kw):
        base = dict(batch=1, layers=2, heads=4, head_dim=128, rank=8, hidden=512, heavy=8, recent=8,
                    max_prompt=64, max_prefill_layers=1, flags=0)
        base.update(kw)
        return B.less_config(**base)
    good = B.less_arena_bytes(cfg())
    assert good > 0 and good % 256 == 0
    assert B.less_state_record_bytes(cfg()) == 16 + 16 * 8 + 2 * 16 * 128 * 2 + 16 * 8 * 4 + 8 * 128 * 4 + 8 * 4
    for bad in (dict(head_dim=32), dict(head_dim=64, flags=16), dict(group=129), dict(group=3, flags=8), dict(rank=4), dict(recent=0), dict(heavy=-1), dict(hidden=500),
                dict(batch=0), dict(max_prefill_layers=3), dict(flags=64), dict(max_prompt=-1),
                dict(heavy=32000, recent=769)):        # more than LESS_MAX_SLOTS = 32768
        assert B.less_arena_bytes(cfg(**bad)) == 0, bad
    assert B.less_arena_bytes(cfg(heavy=32000, recent=768)) > good
    # general shapes: head dimension 64, any number of query heads per KV head up to 128
    assert 0 < B.less_arena_bytes(cfg(head_dim=64)) < good
    assert B.less_arena_bytes(cfg(head_dim=64, group=71)) > B.less_arena_bytes(cfg(head_dim=64))
    assert B.less_arena_bytes(cfg(group=3)) > good
    assert B.less_state_record_bytes(cfg(head_dim=64)) == 16 + 16 * 8 + 2 * 16 * 64 * 2 + 16 * 8 * 4 + 8 * 64 * 4 + 8 * 4
    # arena grows with slots and with the prefill workspace
    assert B.less_arena_bytes(cfg(heavy=80)) > good
    assert B.less_arena_bytes(cfg(max_prompt=4096)) > good
    assert B.less_arena_bytes(cfg(max_prefill_layers=2)) > good


def test_create_rejects_bad_arguments_before_touching_the_device(B):
    c = B.less_config(1, 1, 1, 128, 8, 512, 4, 4, 16, 1, 0)
    w = B.less_weights(256, 256, 256, 256, 256, None)
    rc, _ = B.less_create(c, w, None, 1 << 20)
    assert rc == -2
    rc, _ = B.less_create(c, B.less_weights(256, 256, None, 256, 256, None), 4096, 1 << 30)
    assert rc == -2
    rc, _ = B.less_create(c, B.less_weights(256, 258, 256, 256, 256, None), 4096, 1 << 30)
    assert rc == -3
    rc, _ = B.less_create(c, w, 4096 + 16, 1 << 30)
    assert rc == -3
    rc, _ = B.less_create(c, w, 4096, 1024)
    assert rc == -4
    bad = B.less_config(1, 1, 1, 128, 7, 512, 4, 4, 16, 1, 0)
    rc, _ = B.less_create(bad, w, 4096, 1 << 30)
    assert rc == -1
    assert B.less_strerror(-4) == "arena too small"
    assert B.less_strerror(0) == "ok"


def test_null_context_calls_return_codes(B):
    assert B.less_decode_step(None, None, None, None, None, None, None) == -2
    assert B.less_prefill(None, 0, 1, 0, None, None, None, None, None) == -2
    assert B.less_destroy(None) == -2
    assert B.less_position(None) == -1
    assert B.less_poll_status(None, None) == -2


def test_product_never_imports_the_oracle():
    pkg = os.path.join(ROOT, "paper_2402_09398_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert not re.search(r"^\s*(from|import)\s+oracle\b", text, flags=re.M), f
                assert "oracle/" not in text and "less_oracle" not in text, f


def test_binding_structs_match_the_header(B, tmp_path):
    """The ctypes mirrors of less_config and less_weights have the size and the field offsets a C
    compiler gives the header's structs (a field added on one side only would shift every later one)."""
    import shutil
    import subprocess
    gcc = shutil.which("gcc")
    if gcc is None:
        pytest.skip("no C compiler")
    fields_c = [n for n, _ in B.less_config._fields_]
    fields_w = [n for n, _ in B.less_weights._fields_]
    src = tmp_path / "layout.c"
    lines = ['#include <stdio.h>', '#include <stddef.h>', '#include "less.h"', 'int main(void) {',
             '  printf("%zu %zu\\n", sizeof(less_config), sizeof(less_weights));']
    lines += [f'  printf("%zu\\n", offsetof(less_config, {n}));' for n in fields_c]
    lines += [f'  printf("%zu\\n", offsetof(less_weights, {n}));' for n in fields_w]
    lines += ['  return 0;', '}']
    src.write_text("\n".join(lines))
    exe = tmp_path / "layout"
    subprocess.run([gcc, "-I", os.path.join(ROOT, "include"), str(src), "-o", str(exe)], check=True)
    out = subprocess.run([str(exe)], check=True, capture_output=True, text=True).stdout.split()
    assert int(out[0]) == C.sizeof(B.less_config) and int(out[1]) == C.sizeof(B.less_weights)
    offs = [int(x) for x in out[2:]]
    want = [getattr(B.less_config, n).offset for n in fields_c] + [getattr(B.less_weights, n).offset for n in fields_w]
    assert offs == want
