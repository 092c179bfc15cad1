"""Host-side checks that need no GPU: the shared library builds for sm_100a, loads, exports every
symbol the header declares, and rejects bad arguments before touching the device."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2510_12966_b200 import binding, build
    build.build()
    return binding.load_library()


def declared_symbols():
    text = "".join(open(os.path.join(ROOT, "include", h)).read() for h in sorted(os.listdir(os.path.join(ROOT, "include"))))
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(pyramidsd_[a-z0-9_]+)\s*\(", text)))


def test_header_symbols_are_exported(lib):
    from paper_2510_12966_b200 import binding
    names = declared_symbols()
    assert len(names) >= 10
    for n in names:
        assert hasattr(lib, n), f"{n} declared in include/pyramidsd.h but not exported"
    assert sorted(binding.EXPORTS) == names


def test_struct_layout_matches_header(lib, tmp_path):
    """The argument structs as the C compiler sees them equal their ctypes mirrors: size and the offset of every field."""
    import subprocess
    from paper_2510_12966_b200 import binding
    pairs = (("psd_stage_args", binding.StageArgs), ("psd_pyramid_args", binding.PyramidArgs), ("psd_lmhead_args", binding.LmheadArgs))
    prints = []
    for cname, mirror in pairs:
        prints.append(f'printf("%zu", sizeof({cname}));')
        for fname, _ in mirror._fields_:
            prints.append(f'printf(" %zu", offsetof({cname}, {fname}));')
        prints.append('printf("\\n");')
    src = tmp_path / "sz.c"
    src.write_text('#include "pyramidsd.h"\n#include "pyramidsd_diag.h"\n#include <stdio.h>\n#include <stddef.h>\n'
                   'int main(void){' + "".join(prints) + 'return 0;}\n')
    exe = tmp_path / "sz"
    subprocess.check_call(["gcc", "-std=c99", "-Wall", "-Werror", "-I", os.path.join(ROOT, "include"), str(src), "-o", str(exe)])
    lines = subprocess.check_output([str(exe)]).decode().strip().splitlines()
    for (cname, mirror), line in zip(pairs, lines):
        nums = list(map(int, line.split()))
        assert nums[0] == C.sizeof(mirror), cname
        assert nums[1:] == [getattr(mirror, f).offset for f, _ in mirror._fields_], cname


def test_version_and_status_strings(lib):
    from paper_2510_12966_b200 import binding
    assert "sm_100a" in binding.version()
    assert binding.status_string(0) == "ok" and "invalid" in binding.status_string(-1)


def test_workspace_bytes_is_host_arithmetic(lib):
    from paper_2510_12966_b200 import binding
    small = binding.workspace_bytes(1, 4, 32000, binding.F32)
    big = binding.workspace_bytes(256, 32, 152064, binding.BF16)
    assert 0 < small < big and big >= 256 * 32 * 32
    assert binding.workspace_bytes(1, 33, 100, binding.F32) == 0 and binding.workspace_bytes(1, 4, 0, binding.F32) == 0


def test_invalid_arguments_are_rejected_before_any_launch(lib):
    from paper_2510_12966_b200 import binding
    a = binding.StageArgs()
    assert lib.pyramidsd_verify_stage_ex(C.byref(a)) == binding.ERR_INVALID_ARG          # struct_size 0
    a.struct_size = C.sizeof(binding.StageArgs)
    a.B, a.K, a.V = 1, 1, 0
    assert lib.pyramidsd_verify_stage_ex(C.byref(a)) == binding.ERR_INVALID_ARG          # V < 1
    a.V = 16
    assert lib.pyramidsd_verify_stage_ex(C.byref(a)) == binding.ERR_INVALID_ARG          # NULL outputs
    a.K = 40
    assert lib.pyramidsd_verify_stage_ex(C.byref(a)) == binding.ERR_INVALID_ARG          # K > 32
    a.K, a.V = 1, 1 << 30
    assert lib.pyramidsd_verify_stage_ex(C.byref(a)) == binding.ERR_UNSUPPORTED          # V beyond the limit
    assert lib.pyramidsd_verify_stage_ex(None) == binding.ERR_INVALID_ARG
    assert lib.pyramidsd_verify(None, None, None, None, 1, 4, 8, 100, 1, 0.1, 0.1, 0, 0, 0, None, None, None, None) \
        == binding.ERR_INVALID_ARG                                                        # K_q > K_d, NULLs
    p = binding.PyramidArgs()
    assert lib.pyramidsd_verify_ex(C.byref(p)) == binding.ERR_INVALID_ARG                # struct_size 0
    p.struct_size = C.sizeof(binding.PyramidArgs)
    p.B, p.K_d, p.K_q, p.V, p.mode_q = 0, 8, 4, 100, 7
    assert lib.pyramidsd_verify_ex(C.byref(p)) == binding.ERR_INVALID_ARG                # unknown mode
    p.mode_q, p.schedule = binding.ASSISTED, 9
    assert lib.pyramidsd_verify_ex(C.byref(p)) == binding.ERR_INVALID_ARG                # unknown schedule
    p.schedule, p.seq_index_base = binding.TWO_STAGE_FUSED_ROWS, -1
    assert lib.pyramidsd_verify_ex(C.byref(p)) == binding.ERR_INVALID_ARG                # negative sequence base
    p.seq_index_base = 5
    assert lib.pyramidsd_verify_ex(C.byref(p)) == binding.OK                             # B == 0: a valid empty call
    assert binding.pyramid_workspace_bytes(64, 16, 8, 128256, binding.BF16) == \
        binding.workspace_bytes(64, 16, 128256, binding.BF16) + binding.workspace_bytes(64, 8, 128256, binding.BF16)
    assert binding.pyramid_workspace_bytes(64, 4, 8, 128256, binding.BF16) == 0
    assert lib.pyramidsd_verify_fused_lmhead_ex(None) == binding.ERR_INVALID_ARG
    assert lib.pyramidsd_verify_stage(None, None, None, 0, 4, 100, 0, 0.1, 0, 0, 0, None, None) == binding.OK  # B == 0


def test_missing_library_fails_loudly(tmp_path):
    from paper_2510_12966_b200 import binding
    with pytest.raises(ImportError):
        binding.load_library(str(tmp_path / "libpyramidsd.so"))


def test_product_path_does_not_touch_the_oracle():
    pkg = os.path.join(ROOT, "paper_2510_12966_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text.lower() or f == "workloads.py", f


def test_analytic_throughput_model(lib):
    """Sec. 3.3 formulas against values worked out by hand and their limiting cases."""
    import math
    from paper_2510_12966_b200 import binding
    # beta = 1, ell = 4, draft 100 tok/s, target 20 tok/s: 5 / (0.04 + 0.05) = 55.555...
    assert abs(binding.model_sd_throughput(1.0, 4, 100.0, 20.0) - 5 / 0.09) < 1e-12
    # a draft as slow as the target and always accepted still gains the one free token: (ell+1)/(ell+1) * v
    assert abs(binding.model_sd_throughput(1.0, 7, 30.0, 30.0) - 30.0) < 1e-12
    # nothing accepted: no throughput; the rate is linear in beta
    assert binding.model_sd_throughput(0.0, 4, 100.0, 20.0) == 0.0
    assert abs(binding.model_sd_throughput(0.5, 4, 100.0, 20.0) - 0.5 * 5 / 0.09) < 1e-12
    # pyramid = the pair formula applied twice: inner (0.8, 5, 200, 80) -> 0.8*6/(5/200+1/80) = 128
    inner = binding.model_sd_throughput(0.8, 5, 200.0, 80.0)
    assert abs(inner - 128.0) < 1e-9
    outer = binding.model_psd_throughput(0.8, 5, 200.0, 80.0, 0.9, 10, 25.0)
    assert abs(outer - 0.9 * 11 / (10 / 128.0 + 1 / 25.0)) < 1e-9
    assert math.isnan(binding.model_sd_throughput(1.2, 4, 100.0, 20.0))
    assert math.isnan(binding.model_psd_throughput(0.8, 0, 200.0, 80.0, 0.9, 10, 25.0))
