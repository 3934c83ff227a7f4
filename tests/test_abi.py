"""The C-ABI library loads without a GPU, exports every declared symbol, and validates arguments."""
import ctypes
import os
import re

import pytest

from paper_2006_00441_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "dasgd.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = set(re.findall(r"\b(dasgd_[a-z_0-9]+)\s*\(", text))
    return sorted(names - {"dasgd_status"})      # the return type of the function-pointer typedef, not a function


def test_header_and_library_agree_on_exports():
    names = declared_symbols()
    assert set(names) == set(B.EXPORTS)
    lib = ctypes.CDLL(B._build.LIB)
    for n in names:
        assert hasattr(lib, n), f"libdasgd.so does not export {n}"


def test_version_and_strerror():
    assert re.fullmatch(r"\d+\.\d+", B.dasgd_version())
    assert B._L.dasgd_strerror(B.DASGD_ERR_NO_SLOT) == b"no free snapshot slot"


def _cfg(**kw):
    c = B.dasgd_config()
    c.K, c.tau, c.d, c.P, c.n_slots, c.xi = 4, 2, 1, 64, 1, 0.25
    c.w, c.snap, c.mean = 0x1000, 0x2000, 0x3000
    c.main_stream, c.side_stream = None, 0x10
    for k, v in kw.items():
        setattr(c, k, v)
    return c


@pytest.mark.parametrize("bad,frag", [
    (dict(K=0), "K must"), (dict(P=0), "P must"), (dict(tau=0), "tau must"), (dict(d=-1), "d must"),
    (dict(xi=1.5), "xi must"), (dict(ld=8), "ld must"), (dict(n_slots=0), "n_slots"),
    (dict(d=5, n_slots=2), "n_slots"), (dict(w=None), "must not be NULL"), (dict(momentum=0.9), "needs m"),
    (dict(dtype=1), "needs w_lp"), (dict(dtype=7), "unknown dtype"), (dict(merge_mode=3), "unknown merge_mode"),
    (dict(w=0x1004), "16-byte"), (dict(side_stream=None), "must differ"), (dict(n_stage=3, g_stage=0x4000), "n_stage"),
    (dict(n_stage=1), "given together"), (dict(g_stage=0x4000), "given together"),
    (dict(n_chunks=2), "n_chunks > 1 needs"), (dict(n_chunks=1025, flags=0x8 | 0x4), "n_chunks must"),
    (dict(n_chunks=4, flags=0x8 | 0x4, d=0), "n_chunks > 1 needs"), (dict(n_chunks=-1), "n_chunks must"),
])
def test_init_rejects_bad_configuration_before_touching_cuda(bad, frag):
    with pytest.raises(B.DasgdError) as e:
        B.dasgd_init(_cfg(**bad))
    assert e.value.status == B.DASGD_ERR_INVALID_ARG
    assert frag in str(e.value)


def test_null_context_is_an_error_not_a_crash():
    for fn in (B._L.dasgd_snapshot, B._L.dasgd_average_async, B._L.dasgd_merge, B._L.dasgd_sync, B._L.dasgd_destroy):
        assert fn(None) == B.DASGD_ERR_INVALID_ARG
    assert B._L.dasgd_step(None, None, 0.1) == B.DASGD_ERR_INVALID_ARG


def test_wrapper_refuses_to_run_without_a_gpu():
    import torch
    if torch.cuda.is_available():
        pytest.skip("GPU present")
    with pytest.raises(RuntimeError):
        B.DaSGD(2, 8, 1, 1, 0.25)


def test_header_is_plain_c(tmp_path):
    """include/dasgd.h must compile as C99 on its own and every declared function must be linkable from C."""
    import subprocess
    src = tmp_path / "use_dasgd.c"
    calls = "\n".join(f"  (void)&{n};" for n in declared_symbols())
    src.write_text('#include "dasgd.h"\n#include <stddef.h>\nint main(void) {\n  dasgd_config c; c.K = 1; (void)c;\n'
                   + calls + "\n  return (int)sizeof(dasgd_config) == 0;\n}\n")
    exe = tmp_path / "use_dasgd"
    subprocess.run(["gcc", "-std=c99", "-Wall", "-Werror", "-pedantic", "-I", os.path.join(ROOT, "include"), str(src),
                    B._build.LIB, "-Wl,-rpath," + os.path.dirname(B._build.LIB), "-o", str(exe)], check=True)
    subprocess.run([str(exe)], check=True)


def test_config_struct_layout_matches_the_binding(tmp_path):
    """sizeof and field offsets of dasgd_config as the C compiler sees them == the ctypes mirror."""
    import subprocess
    fields = [f[0] for f in B.dasgd_config._fields_]
    body = "\n".join(f'  printf("{f} %zu\\n", offsetof(dasgd_config, {f}));' for f in fields)
    src = tmp_path / "layout.c"
    src.write_text('#include "dasgd.h"\n#include <stddef.h>\n#include <stdio.h>\nint main(void) {\n'
                   + body + '\n  printf("sizeof %zu\\n", sizeof(dasgd_config));\n  return 0;\n}\n')
    exe = tmp_path / "layout"
    subprocess.run(["gcc", "-std=c99", "-I", os.path.join(ROOT, "include"), str(src), "-o", str(exe)], check=True)
    out = dict(line.split() for line in subprocess.run([str(exe)], check=True, capture_output=True, text=True).stdout.splitlines())
    for f in fields:
        assert int(out[f]) == getattr(B.dasgd_config, f).offset, f
    assert int(out["sizeof"]) == ctypes.sizeof(B.dasgd_config)
