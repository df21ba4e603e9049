"""CPU-side checks of the C ABI: the library builds, loads, exports every symbol the
header declares, agrees with the binding on struct layout, validates arguments, and
refuses to run without a CUDA device (there is no CPU path)."""
import ctypes as C
import os
import re
import subprocess
import tempfile

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "pbt.h")


@pytest.fixture(scope="module")
def pkg():
    from paper_1711_09846_b200.build import build
    build()
    import paper_1711_09846_b200 as p
    p.load_library()
    return p


def _declared():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(pbt_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(pkg):
    lib = pkg.load_library()
    names = _declared()
    assert len(names) >= 20
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(pkg.EXPORTS) == [n for n in names if n in pkg.EXPORTS]
    assert set(names) == set(pkg.EXPORTS)


def test_struct_layout_matches_the_header(pkg):
    from paper_1711_09846_b200 import binding as B
    src = r'''
#include <stdio.h>
#include <stddef.h>
#include "pbt.h"
int main(void) {
  printf("%zu %zu %zu %zu %zu %zu %zu %zu\n", sizeof(pbt_spec), offsetof(pbt_spec, widths), offsetof(pbt_spec, slot_lr),
         offsetof(pbt_spec, const_lr), offsetof(pbt_spec, clamp_hi), sizeof(pbt_data), sizeof(pbt_state_view),
         offsetof(pbt_spec, toy_theta0));
  return 0;
}'''
    with tempfile.TemporaryDirectory() as d:
        c = os.path.join(d, "t.c")
        open(c, "w").write(src)
        exe = os.path.join(d, "t")
        subprocess.run(["gcc", "-I", os.path.join(ROOT, "include"), c, "-o", exe], check=True)
        got = [int(x) for x in subprocess.run([exe], capture_output=True, text=True, check=True).stdout.split()]
    S = B.PbtSpec
    assert got == [C.sizeof(S), S.widths.offset, S.slot_lr.offset, S.const_lr.offset, S.clamp_hi.offset,
                   C.sizeof(B.PbtData), C.sizeof(B.PbtStateView), S.toy_theta0.offset]


def test_param_counts_and_workspace_sizes(pkg):
    from workloads import get_config
    expect = {"c1": 2, "c2": 394753, "c3": 1863690, "c4": 296962 + 264705, "c5": 14687232}
    lib = pkg.load_library()
    for name, p in expect.items():
        cfg = get_config(name)
        assert pkg.param_count(cfg) == p
        spec = pkg.spec_from_config(cfg)
        n = C.c_size_t(0)
        assert lib.pbt_query_workspace(C.byref(spec), C.byref(n)) == 0
        if name != "c1":
            # at least master + two moments (or momentum) + gradient per member
            slabs = 4 if cfg.optimizer == "adam" else 3
            assert n.value >= cfg.n_members * p * 4 * slabs
            assert n.value < 40e9
        assert n.value % 256 == 0


def test_invalid_specs_are_rejected_with_a_message(pkg):
    from workloads import get_config
    lib = pkg.load_library()
    n = C.c_size_t(0)
    for mutate, code in ((lambda s: setattr(s, "n_members", 0), 1),
                         (lambda s: setattr(s, "nh", 99), 1),
                         (lambda s: setattr(s, "slot_lr", 7), 1),
                         (lambda s: setattr(s, "dtype", 0), 2),
                         (lambda s: setattr(s, "optimizer", 9), 2),
                         (lambda s: setattr(s, "pool_rows", 1), 1),
                         (lambda s: setattr(s, "trunc_den", 0), 1)):
        spec = pkg.spec_from_config(get_config("c2_mini"))
        mutate(spec)
        assert lib.pbt_query_workspace(C.byref(spec), C.byref(n)) == code
        assert len(lib.pbt_last_error(None)) > 0
    assert lib.pbt_query_workspace(None, C.byref(n)) == 1
    assert lib.pbt_step(None, 1) == 1


def test_no_cpu_fallback(pkg):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a CUDA device is present")
    from workloads import get_config, make_inputs
    cfg = get_config("c1")
    with pytest.raises(RuntimeError):
        pkg.Population(cfg, make_inputs(cfg))
    lib = pkg.load_library()
    spec = pkg.spec_from_config(cfg)
    handle = C.c_void_p(None)
    buf = (C.c_char * 8192)()
    base = (C.addressof(buf) + 255) // 256 * 256
    h0 = (C.c_double * 4)(1, 0, 0, 1)
    rc = lib.pbt_create(C.byref(handle), C.byref(spec), h0, 0, None, C.c_void_p(base), 4096, None)
    assert rc == 4 and not handle.value          # PBT_ERR_CUDA, no handle
    assert b"no CPU path" in lib.pbt_last_error(None)


def test_product_code_never_touches_the_oracle():
    pk = os.path.join(ROOT, "paper_1711_09846_b200")
    for dirpath, _, files in os.walk(pk):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text, f
    for dirpath, _, files in os.walk(os.path.join(ROOT, "oracle")):
        for f in files:
            if f.endswith(".py"):
                text = open(os.path.join(dirpath, f)).read()
                assert "paper_1711_09846_b200" not in text and "ctypes" not in text, f
