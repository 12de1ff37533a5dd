"""Host-only checks of the C ABI: the library loads without a GPU, exports every symbol the
header declares, its structs have the layout the binding assumes, and host-side argument
checks answer without touching a device."""
import ctypes as C
import os
import re
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "td.h")


@pytest.fixture(scope="module")
def td():
    from paper_2507_19017_b200 import build, binding
    build.build()
    return binding


def declared_functions():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(td_[a-z_]+)\s*\(", text)))


def test_header_declares_what_the_binding_lists(td):
    assert declared_functions() == sorted(td.EXPORTS)


def test_library_exports_every_declared_symbol(td):
    lib = C.CDLL(td.lib_path())
    for name in declared_functions():
        assert hasattr(lib, name), name


def test_struct_layouts_match_the_header(td, tmp_path):
    src = tmp_path / "sizes.c"
    src.write_text(
        '#include <stdio.h>\n#include <stddef.h>\n#include "td.h"\n'
        "int main(void){printf(\"%zu %zu %zu %zu %zu %zu %zu %zu %zu %zu\\n\", sizeof(td_column),"
        "sizeof(td_consumer), sizeof(td_config), sizeof(td_result), sizeof(td_get_out), sizeof(td_stats),"
        "offsetof(td_get_out, col), offsetof(td_get_out, advantages), offsetof(td_get_out, scratch),"
        "offsetof(td_config, reward_column)); return 0;}\n")
    exe = tmp_path / "sizes"
    subprocess.check_call(["gcc", "-std=c11", "-I", os.path.join(ROOT, "include"), "-o", str(exe), str(src)])
    got = list(map(int, subprocess.check_output([str(exe)]).split()))
    want = [C.sizeof(td.TdColumn), C.sizeof(td.TdConsumer), C.sizeof(td.TdConfig), C.sizeof(td.TdResult),
            C.sizeof(td.TdGetOut), C.sizeof(td.TdStats), td.TdGetOut.col.offset,
            td.TdGetOut.advantages.offset, td.TdGetOut.scratch.offset, td.TdConfig.reward_column.offset]
    assert got == want


def _cfg(td, **kw):
    args = dict(G=8, N=4, S=2, columns=[("i32", "prompt", 0), ("i32", "response", 0), ("f32", "scalar", 0)],
                consumers=[(3, 3, False), (7, 7, True)], prompt_cap=128, response_cap=1024,
                reward_column=2)
    args.update(kw)
    return td.make_config(**args)


def test_query_workspace_needs_no_gpu_and_grows_with_capacity(td):
    cfg, keep = _cfg(td)
    small = td.query_workspace(cfg)
    cfg2, keep2 = _cfg(td, response_cap=2048)
    big = td.query_workspace(cfg2)
    assert small % 256 == 0 and big - small == 2 * 1024 * 4      # one response column, two shards
    assert small >= 2 * (128 + 1024) * 4


@pytest.mark.parametrize("bad", [
    dict(S=3),                                   # shards must divide prompts
    dict(consumers=[(1, 3, False)]),             # out outside need
    dict(consumers=[(3, 3, True)]),              # advantage without the reward column
    dict(reward_column=0, consumers=[(7, 7, True)]),   # reward column is not an f32 scalar
    dict(G=0),
    dict(S=512, G=512),
])
def test_invalid_configurations_are_refused(td, bad):
    cfg, keep = _cfg(td, **bad)
    out = C.c_size_t(0)
    assert td.lib().td_query_workspace(C.byref(cfg), C.byref(out)) == td.EINVAL


def test_create_reports_workspace_and_argument_errors_before_any_cuda_call(td):
    cfg, keep = _cfg(td)
    h = C.c_void_p()
    need = td.query_workspace(cfg)
    assert td.lib().td_create(C.byref(cfg), None, need, C.byref(h)) == td.EINVAL
    assert td.lib().td_create(C.byref(cfg), 4096, need - 1, C.byref(h)) == td.EWORKSPACE
    assert td.lib().td_create(C.byref(cfg), 4096 + 8, need, C.byref(h)) == td.EWORKSPACE   # misaligned
    assert td.lib().td_strerror(td.EWORKSPACE).decode().startswith("workspace")
    assert td.lib().td_put(None, 0, None, 1, None, None, 0, None) == td.EINVAL
    assert td.lib().td_get(None, 0, 8, None, None) == td.EINVAL
    assert td.lib().td_launch_count(None) == 0
    assert td.lib().td_put_back(None, None, 8, None, 0, None) == td.EINVAL
    assert td.lib().td_put_back_many(None, None, 0, None) == td.EINVAL
    assert td.lib().td_get_many(None, None, None) == td.EINVAL
    assert td.lib().td_get_many_host(None, None, None, 0, None, 0, None) == td.EINVAL
    assert td.lib().td_put_many_host(None, None, 0, None, 0, None) == td.EINVAL
    assert td.lib().td_get_many_host_stage_bytes(None) == 0
    rep = td.TdValidateReport()
    assert td.lib().td_debug_validate(None, None, C.byref(rep)) == td.EINVAL


def test_create_fails_loudly_without_a_device(td):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    cfg, keep = _cfg(td)
    h = C.c_void_p()
    assert td.lib().td_create(C.byref(cfg), 256 * 1024, td.query_workspace(cfg), C.byref(h)) == td.ECUDA
    assert not h.value


def test_missing_library_raises(td, monkeypatch):
    monkeypatch.setattr(td, "_lib", None)
    monkeypatch.delenv("TD_LIB_PATH", raising=False)
    monkeypatch.setattr(td._build, "LIB_PATH", "/nonexistent/libtd.so")
    with pytest.raises(RuntimeError):
        td.lib()


def test_build_with_nvtx_ranges_exports_the_same_symbols(td, tmp_path):
    """-DTD_NVTX wraps the public calls in named ranges for timeline tools; the build must succeed
    against the toolkit's header-only nvtx3 and change nothing about the ABI."""
    from paper_2507_19017_b200 import build as b
    out = str(tmp_path / "libtd_nvtx.so")
    cmd = [b._nvcc()] + b.NVCC_FLAGS + ["-DTD_NVTX", "-o", out] + [os.path.join(b.CSRC, s) for s in b.SOURCES] + ["-ldl"]
    env = {k: v for k, v in os.environ.items() if k != "LD_PRELOAD"}      # the compiler runs without any preloaded runtime
    res = subprocess.run(cmd, capture_output=True, text=True, timeout=900, env=env)
    assert res.returncode == 0, res.stderr[-2000:]
    lib = C.CDLL(out)
    for name in declared_functions():
        assert hasattr(lib, name), name
    lib.td_strerror.restype = C.c_char_p
    assert lib.td_strerror(0) == b"ok"
