"""Host-side checks that need no GPU: the C-ABI library loads, exports every symbol the header
declares, and validates arguments before touching CUDA."""
import ctypes as C
import os
import re

import pytest

from paper_2608_14624_b200 import binding as cs
from paper_2608_14624_b200 import build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build_library()
    return cs.lib()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "cachescout.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(cs_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_symbols()
    assert len(names) >= 17
    for name in names:
        assert hasattr(lib, name), name
    assert set(names) == set(cs.EXPORTS)
    assert cs.cs_version() >= 100


def test_workspace_sizing_and_param_validation(lib):
    p = cs.make_params(n_agents=12, n_chains=64, max_blocks=80000)
    small = cs.cs_workspace_bytes(p)
    big = cs.cs_workspace_bytes(cs.make_params(n_agents=256, n_chains=16, max_blocks=1_000_000))
    # 32 B of select scratch per entry for each of the three selects that may run side by side
    assert 80000 * 96 <= small < 80000 * 100 + (1 << 20)
    assert 96_000_000 <= big < 100_000_000
    huge = cs.cs_workspace_bytes(cs.make_params(n_agents=256, n_chains=16, max_blocks=64_000_000))
    assert 64_000_000 * 32 <= huge < 64_000_000 * 33 + (32 << 20)      # beyond 4,194,304 entries: one full-size region only
    for bad in (dict(n_agents=0), dict(n_agents=2000), dict(n_agents=4, eps=0.0), dict(n_agents=4, delta=0.0),
                dict(n_agents=4, lam=-1.0), dict(n_agents=4, e_max=0), dict(n_agents=4, block_tokens=0),
                dict(n_agents=4, max_blocks=0), dict(n_agents=4, n_chains=0), dict(n_agents=4, tau=float("nan"))):
        with pytest.raises(cs.CacheScoutError) as e:
            cs.cs_workspace_bytes(cs.make_params(**bad))
        assert e.value.code == cs.CS_EINVAL
    n = C.c_size_t()
    assert lib.cs_workspace_bytes(None, C.byref(n)) == cs.CS_EINVAL
    assert lib.cs_workspace_bytes(C.byref(p), None) == cs.CS_EINVAL


def test_null_context_is_rejected_without_cuda(lib):
    assert lib.cs_destroy(None) == cs.CS_EINVAL
    assert lib.cs_observe_invocations(None, None, None, None, 0, None) == cs.CS_EINVAL
    assert lib.cs_launch_count(None, None) == cs.CS_EINVAL
    assert lib.cs_strerror(cs.CS_ECAPACITY).decode().startswith("size beyond")
    assert lib.cs_strerror(-99).decode() == "unknown error"
    ctx = C.c_void_p()
    p = cs.make_params(n_agents=4)
    assert lib.cs_create(C.byref(p), None, 1 << 20, None, C.byref(ctx)) == cs.CS_EINVAL        # NULL workspace
    assert lib.cs_create(C.byref(p), 256 + 8, 1 << 20, None, C.byref(ctx)) == cs.CS_EINVAL     # misaligned
    assert lib.cs_create(C.byref(p), 4096, 16, None, C.byref(ctx)) == cs.CS_ECAPACITY          # too small


def test_product_path_has_no_cpu_fallback():
    import torch
    if torch.cuda.is_available():
        pytest.skip("GPU present")
    with pytest.raises(RuntimeError):
        cs.CacheScout(cs.make_params(n_agents=4), "cuda:0")


def test_header_is_plain_c_and_cxx():
    """The boundary header must be usable from C (C99) and from C++ without anything else included."""
    import shutil
    import subprocess
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    src = '#include "cachescout.h"\nint use(void) { cs_params p = {0}; cs_step_io io = {0}; return (int)p.n_agents + (int)io.now; }\n'
    for cc, std, lang in (("gcc", "-std=c99", "c"), ("g++", "-std=c++17", "c++")):
        if shutil.which(cc) is None:
            pytest.skip("no %s here" % cc)
        r = subprocess.run([cc, std, "-Wall", "-Werror", "-pedantic", "-fsyntax-only", "-I", os.path.join(root, "include"),
                            "-x", lang, "-"], input=src, capture_output=True, text=True)
        assert r.returncode == 0, r.stderr
