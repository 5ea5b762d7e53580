"""Host-only checks of the C ABI: the library loads, exports every symbol the header declares, and
rejects bad arguments before touching a device.  No GPU needed."""
import ctypes as C
import os
import re

import numpy as np
import pytest

import __graft_entry__ as entry

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def api():
    entry.build()
    from paper_1905_10395_b200 import api as a
    return a


def test_library_exports_every_declared_symbol(api):
    with open(os.path.join(ROOT, "include", "lsgd.h")) as fh:
        header = fh.read()
    declared = set(re.findall(r"LSGD_API\s+[\w\s\*]+?\b(lsgd_\w+)\s*\(", header))
    assert {"lsgd_create", "lsgd_grad", "lsgd_elect", "lsgd_step", "lsgd_destroy"} <= declared
    L = api.lib()
    for name in declared:
        assert hasattr(L, name), name


def test_struct_layout_matches_header(api, tmp_path):
    # the header compiles as plain C, and the binding's structs have the sizes the C compiler gives
    import subprocess
    src = tmp_path / "sz.c"
    src.write_text('#include <stdio.h>\n#include "lsgd.h"\nint main(void){printf("%zu %zu %zu %zu %zu %zu\\n",'
                   'sizeof(lsgd_config),sizeof(lsgd_quadratic_desc),sizeof(lsgd_matcomp_desc),'
                   'sizeof(lsgd_mlp_desc),sizeof(lsgd_psd_desc),sizeof(lsgd_bgemm_desc));return 0;}\n')
    exe = tmp_path / "sz"
    subprocess.run(["gcc", "-std=c99", "-Wall", "-Werror", "-I", os.path.join(ROOT, "include"), str(src), "-o",
                    str(exe)], check=True)
    sizes = [int(v) for v in subprocess.run([str(exe)], capture_output=True, text=True, check=True).stdout.split()]
    assert sizes == [C.sizeof(api.Config), C.sizeof(api.QuadraticDesc), C.sizeof(api.MatcompDesc),
                     C.sizeof(api.MlpDesc), C.sizeof(api.PsdDesc), C.sizeof(api.BgemmDesc)]


def _cfg(api, **over):
    kw = dict(P=4, G=2, group_of=np.array([0, 0, 1, 1]), d=100, ld=128, eta=0.1, lambda_l=0.1, lambda_g=0.1, tau=1,
              objective=api.OBJ_EXTERNAL, x=4096, g=8192)
    kw.update(over)
    return api.make_config(**kw)


@pytest.mark.parametrize("over,status", [
    (dict(P=0), 1), (dict(tau=0), 1), (dict(d=200), 1), (dict(eta=float("nan")), 1),
    (dict(G=5), 2), (dict(G=0), 2), (dict(group_of=np.array([0, 0, 0, 0])), 2), (dict(group_of=np.array([0, 1, 2, 1])), 2),
    (dict(ld=100), 3), (dict(x=4100), 3), (dict(g=8200), 3),
    (dict(x=None), 1), (dict(g=None), 1), (dict(objective=9), 1), (dict(arithmetic=7), 1),
    (dict(objective=1), 1),                      # quadratic without its descriptor
])
def test_create_rejects_bad_arguments_on_the_host(api, over, status):
    cfg, keep = _cfg(api, **over)
    h = C.c_void_p(123)
    s = api.lib().lsgd_create(C.byref(cfg), C.byref(h))
    assert s == status, api.status_string(s)
    assert h.value is None


def test_create_rejects_shapes_beyond_the_documented_capacities(api):
    # population too large for the group tables of the register-staged pull kernel (P + 2 G + 2 > 12288)
    P = 4096
    cfg, keep = _cfg(api, P=P, G=P, group_of=np.arange(P))
    h = C.c_void_p()
    assert api.lib().lsgd_create(C.byref(cfg), C.byref(h)) == api.ERR_UNSUPPORTED
    # matrix-completion batch beyond the range of the fixed-point accumulator
    desc = api.MatcompDesc(10, 10, 5, 50, 4096, 4096, 4096, (1 << 15) + 1, 8, 4096, None, 0)
    cfg, keep = _cfg(api, d=100, objective=api.OBJ_MATCOMP, desc=desc)
    assert api.lib().lsgd_create(C.byref(cfg), C.byref(h)) == api.ERR_UNSUPPORTED


def test_caller_owned_scratch_is_validated_on_the_host(api):
    P, ld = 4, 128
    need = api.matcomp_scratch_bytes(P, ld)
    assert need == 8 * P * ld
    h = C.c_void_p()
    for scratch, nbytes, status in [(4096 + 8, need, api.ERR_ALIGNMENT), (4096, need - 1, api.ERR_INVALID_ARG)]:
        desc = api.MatcompDesc(10, 10, 5, 50, 4096, 4096, 4096, 16, 8, 4096, scratch, nbytes)
        cfg, keep = _cfg(api, d=100, objective=api.OBJ_MATCOMP, desc=desc)
        assert api.lib().lsgd_create(C.byref(cfg), C.byref(h)) == status
    assert api.psd_scratch_bytes(100, 8, 100000) == 0                    # large ranks need none
    need = api.psd_scratch_bytes(10, 4, 128)                             # two fp64 partial gradients at small rank
    assert need == 16 * 4 * 128
    desc = api.PsdDesc(10, 10, 4096, 8192, need - 8)
    cfg, keep = _cfg(api, d=100, objective=api.OBJ_PSD_COMPLETION, desc=desc)
    assert api.lib().lsgd_create(C.byref(cfg), C.byref(h)) == api.ERR_INVALID_ARG


def test_device_flag_bits_match_the_header(api):
    with open(os.path.join(ROOT, "include", "lsgd.h")) as fh:
        header = fh.read()
    bits = {m.group(1): int(m.group(2)) for m in re.finditer(r"#define LSGD_DEVFLAG_(\w+) (\d+)u", header)}
    assert bits == {"BAD_LEADER": api.DEVFLAG_BAD_LEADER, "WAIT_TIMEOUT": api.DEVFLAG_WAIT_TIMEOUT,
                    "BAD_INDEX": api.DEVFLAG_BAD_INDEX, "OVERFLOW": api.DEVFLAG_OVERFLOW}


def test_struct_size_is_checked(api):
    cfg, keep = _cfg(api)
    cfg.struct_size = 8
    h = C.c_void_p()
    assert api.lib().lsgd_create(C.byref(cfg), C.byref(h)) == api.ERR_INVALID_ARG


def test_null_handles(api):
    L = api.lib()
    assert L.lsgd_grad(None, None) == api.ERR_INVALID_ARG
    assert L.lsgd_elect(None, None) == api.ERR_INVALID_ARG
    assert L.lsgd_step(None) == api.ERR_INVALID_ARG
    assert L.lsgd_destroy(None) == api.OK
    assert api.status_string(api.ERR_STATE)
    out = (C.c_int32 * 3)()
    assert L.lsgd_shard_best_key(None, 1, None, None) == api.ERR_INVALID_ARG
    assert L.lsgd_shard_pick_global(None, None, 1, 0, 0, out) == api.ERR_INVALID_ARG
    assert L.lsgd_selftest_wait_timeout(None, 0, 1000, out) == api.ERR_INVALID_ARG
    assert L.lsgd_mlp_get_activations(None, None, None) == api.ERR_INVALID_ARG
    assert L.lsgd_set_leaders(None, None, 0) == api.ERR_INVALID_ARG
    assert L.lsgd_center(None, None) == api.ERR_INVALID_ARG
    assert api.matcomp_scratch_bytes(0, 32) == 0 and api.psd_scratch_bytes(0, 1, 32) == 0


def test_mlp_offsets_match_the_input_generator_layout(api):
    from paper_1905_10395_b200 import inputs
    for dims in [(784, 1024, 1024, 10), (5, 4, 4, 3), (33, 65, 17, 9)]:
        segs, d = inputs.mlp_layout(dims)
        w, b, dd = api.mlp_param_offsets(dims)
        assert dd == d and w == [s["w"] for s in segs] and b == [s["b"] for s in segs]


def test_no_device_is_an_error_not_a_fallback(api):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    cfg, keep = _cfg(api)
    h = C.c_void_p()
    assert api.lib().lsgd_create(C.byref(cfg), C.byref(h)) == api.ERR_CUDA
