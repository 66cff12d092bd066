"""Host-side checks of the C ABI: the library loads, exports every declared symbol, and
rejects bad calls without a GPU."""
import ctypes
import os
import re

import pytest

import paper_2009_02701_b200 as hp
from paper_2009_02701_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "hpsgd.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(hpsgd_[a-z_0-9]+)\s*\(", text)))


def test_library_builds_and_exports_every_declared_symbol():
    path = build.build()
    lib = ctypes.CDLL(path)
    names = declared_symbols()
    assert len(names) >= 20
    for name in names:
        assert hasattr(lib, name), "%s is declared in hpsgd.h but not exported" % name
    assert sorted(binding.SIGNATURES) == names, "binding and header disagree"


def test_layout_is_pure_host_code():
    pad, off = hp.hpsgd_layout_padded([5, 64, 33, 1])
    assert (pad, off) == (192, [0, 32, 96, 160])
    with pytest.raises(hp.HpsgdError) as err:
        hp.hpsgd_layout_padded([5, 0])
    assert err.value.code == hp.HPSGD_E_BADARG
    import workloads
    for name in workloads.names():
        lay = workloads.get(name).layout
        pad, off = hp.hpsgd_layout_padded(list(lay.sizes))
        assert pad == lay.P_pad and off == lay.offsets


def test_arena_size_formula():
    # w + D + K replicas (+ K momenta), rows padded to 256 bytes, plus table and slot maps
    P_pad, K = 1_048_576, 4
    plain = hp.hpsgd_arena_bytes(P_pad, K, 0, 0)
    mom = hp.hpsgd_arena_bytes(P_pad, K, hp.HPSGD_ARENA_MOMENTUM, 0)
    assert mom - plain == K * P_pad * 4
    assert plain >= (K + 2) * P_pad * 4
    assert hp.hpsgd_arena_bytes(P_pad, K, 0, 30_000) - plain >= 30_000 * 4 * K
    assert hp.hpsgd_arena_bytes(0, K, 0, 0) == 0


def test_calls_before_init_fail_cleanly():
    hp.hpsgd_destroy()
    for call in (hp.hpsgd_sync_merge, hp.hpsgd_synchronize, lambda: hp.hpsgd_local_step(0, 256),
                 hp.hpsgd_get_global, lambda: hp.hpsgd_set_option(hp.HPSGD_OPT_CHUNKS, 2)):
        with pytest.raises(hp.HpsgdError) as err:
            call()
        assert err.value.code == hp.HPSGD_E_STATE
    assert "hpsgd_init" in hp.last_error()
    assert hp.hpsgd_launch_count() == 0


def test_init_validates_arguments_before_touching_the_device():
    hp.hpsgd_destroy()
    for args in ((0, 4, 0.1, 0.0, 1), (100, 0, 0.1, 0.0, 1), (100, 4, -0.1, 0.0, 1), (100, 4, 0.1, 1.0, 1),
                 (100, 4, 0.1, -0.5, 1), (100, 300, 0.1, 0.0, 1)):
        with pytest.raises(hp.HpsgdError) as err:
            hp.hpsgd_init(*args)
        assert err.value.code == hp.HPSGD_E_BADARG
    hp.hpsgd_set_layout([10, 20])
    with pytest.raises(hp.HpsgdError) as err:
        hp.hpsgd_init(31, 2, 0.1, 0.0, 1)
    assert err.value.code == hp.HPSGD_E_BADARG
    hp.hpsgd_destroy()
    with pytest.raises(hp.HpsgdError):
        hp.hpsgd_bind(128, 1024, None, None)        # not 256-byte aligned
    with pytest.raises(hp.HpsgdError):
        hp.hpsgd_bind(None, 0, 1, None)             # one stream only


def test_no_cpu_fallback_without_a_device():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a CUDA device is present")
    hp.hpsgd_destroy()
    with pytest.raises(hp.HpsgdError) as err:
        hp.hpsgd_init(1000, 4, 0.1, 0.0, 1)
    assert err.value.code == hp.HPSGD_E_CUDA


def test_product_code_never_touches_the_oracle():
    pkg = os.path.join(ROOT, "paper_2009_02701_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text, "%s mentions the oracle" % f
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith((".py", ".cpp")):
            text = open(os.path.join(ROOT, "oracle", f)).read()
            assert "paper_2009_02701_b200" not in text and "libhpsgd.so" not in text


def test_header_is_plain_c(tmp_path):
    """The boundary is a C ABI: the header must compile as C99 and as C++ with no other include."""
    import subprocess
    src = tmp_path / "use_header.c"
    src.write_text('#include "hpsgd.h"\n'
                   'int probe(void) { hpsgd_grad_desc d = {0, 0, 0, 0}; (void)d; '
                   'return (int)sizeof(hpsgd_status) + HPSGD_OPT_FUSE + HPSGD_NOALLOC_MAX_ROWS; }\n')
    inc = os.path.join(ROOT, "include")
    subprocess.run(["gcc", "-std=c99", "-Wall", "-Werror", "-pedantic", "-fsyntax-only", "-I", inc, str(src)], check=True)
    subprocess.run(["g++", "-std=c++17", "-Wall", "-Werror", "-fsyntax-only", "-x", "c++", "-I", inc, str(src)], check=True)


def test_layout_matches_the_workload_helper_on_random_size_lists():
    """Two independent implementations of the flat layout (the library's and the input module's)."""
    import numpy as np
    from workloads.configs import Layout
    rng = np.random.default_rng(3)
    for _ in range(200):
        sizes = [int(x) for x in rng.integers(1, 5000, size=int(rng.integers(1, 40)))]
        pad, off = hp.hpsgd_layout_padded(sizes)
        lay = Layout(sizes)
        assert (pad, off) == (lay.P_pad, lay.offsets)
        assert all(o % 32 == 0 for o in off) and pad % 32 == 0
        assert all(off[i + 1] - off[i] >= sizes[i] for i in range(len(sizes) - 1))
        # the arena holds at least w, D and K rows of P_pad floats (+ K more with momentum or the
        # pipelined schedule), whatever the padding
        K = int(rng.integers(1, 20))
        base = hp.hpsgd_arena_bytes(pad, K, 0, 0)
        assert base >= (K + 2) * pad * 4
        assert hp.hpsgd_arena_bytes(pad, K, hp.HPSGD_ARENA_MOMENTUM, 0) - base >= K * pad * 4
        assert hp.hpsgd_arena_bytes(pad, K, hp.HPSGD_ARENA_PIPELINE, 0) - base >= (K + 1) * pad * 4
        assert hp.hpsgd_arena_bytes(pad, K, 0, 1000) - base >= 1000 * 4 * K
