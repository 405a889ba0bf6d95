"""Host-only checks of the C-ABI library: it loads, exports every declared symbol, validates
arguments before touching the device, and its built-in level table equals the oracle's."""
import ctypes
import os
import re

import numpy as np
import pytest

import oracle

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2407_17029_b200 import build
    return ctypes.CDLL(build.build())


def declared_symbols():
    hdr = open(os.path.join(ROOT, "include", "qblora.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    return sorted(set(re.findall(r"\b(qa?blora_[a-z_0-9]+)\s*\(", hdr)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_symbols()
    assert {"qblora_quantize_blockwise", "qblora_linear_fwd", "qblora_linear_bwd", "qablora_merge",
            "qablora_lowbit_gemm"} <= set(names)
    for n in names:
        assert getattr(lib, n) is not None


def test_binding_lists_the_same_symbols():
    from paper_2407_17029_b200 import binding
    assert set(binding.EXPORTS) <= set(declared_symbols())


def test_default_table_equals_oracle_bit_for_bit(lib):
    buf = (ctypes.c_float * 16)()
    assert lib.qblora_default_code_table(buf) == 0
    got = np.array(list(buf), dtype=np.float32)
    assert np.array_equal(got.view(np.uint32), oracle.default_code_table().view(np.uint32))


def test_status_strings(lib):
    lib.qblora_status_string.restype = ctypes.c_char_p
    assert lib.qblora_status_string(0) == b"ok"
    assert len({lib.qblora_status_string(i) for i in range(6)}) == 6


def test_argument_validation_happens_on_the_host(lib):
    from paper_2407_17029_b200 import binding as qb
    # null weight
    assert lib.qblora_linear_fwd(None, None, None, ctypes.c_int64(1), None, 1, None, ctypes.c_size_t(0), None) == qb.ERR_INVALID_ARG
    # geometry that does not divide
    code = (ctypes.c_float * 16)(*[float(x) for x in oracle.default_code_table()])
    fake = ctypes.c_void_p(0x1000)
    rc = lib.qblora_quantize_blockwise(fake, 0, 4, 96, 64, 1, 0, code, fake, fake, None, None)
    assert rc == qb.ERR_INVALID_ARG
    # misaligned pointer
    rc = lib.qblora_quantize_blockwise(ctypes.c_void_p(0x1004), 0, 4, 128, 64, 1, 0, code, fake, fake, None, None)
    assert rc == qb.ERR_INVALID_ARG
    # non-monotone table
    bad = (ctypes.c_float * 16)(*([0.0] * 16))
    rc = lib.qblora_quantize_blockwise(fake, 0, 4, 128, 64, 1, 0, bad, fake, fake, None, None)
    assert rc == qb.ERR_INVALID_ARG


def test_workspace_bytes_and_merge_alignment_rule(lib):
    from paper_2407_17029_b200 import binding as qb
    lib.qblora_workspace_bytes.restype = ctypes.c_size_t
    q = qb._CQWeight()
    q.d_in, q.d_out, q.block_in, q.block_out, q.qfmt = 4096, 4096, 64, 1, 1
    q.codes = q.alpha = q.beta = 0x1000
    a = qb._CAdapter()
    a.lambda_in, a.lambda_out, a.rank, a.scaling = 64, 8, 256, 1.0
    a.A = a.B = 0x1000
    for op in (qb.OP_LINEAR_FWD, qb.OP_LINEAR_BWD, qb.OP_MERGE, qb.OP_LOWBIT_GEMM):
        n = lib.qblora_workspace_bytes(op, ctypes.byref(q), ctypes.byref(a), ctypes.c_int64(2048))
        assert n >= 256
    assert lib.qblora_workspace_bytes(qb.OP_QUANTIZE, ctypes.byref(q), None, ctypes.c_int64(0)) == 0
    # workspace too small is reported before any launch
    rc = lib.qablora_merge(ctypes.byref(q), ctypes.byref(a), ctypes.c_void_p(0x1000), ctypes.c_void_p(0x1000),
                           ctypes.c_size_t(16), None)
    assert rc == qb.ERR_WORKSPACE
    # a 64-wide quantization block cannot sit inside a 4-wide tile of the dense update
    a.lambda_in, a.lambda_out = 4, 4
    rc = lib.qablora_merge(ctypes.byref(q), ctypes.byref(a), ctypes.c_void_p(0x1000), ctypes.c_void_p(0x1000),
                           ctypes.c_size_t(1 << 30), None)
    assert rc == qb.ERR_INVALID_ARG
    # code-table weights cannot be merged into
    q.qfmt = 0
    a.lambda_in, a.lambda_out = 64, 8
    rc = lib.qablora_merge(ctypes.byref(q), ctypes.byref(a), ctypes.c_void_p(0x1000), ctypes.c_void_p(0x1000),
                           ctypes.c_size_t(1 << 30), None)
    assert rc == qb.ERR_INVALID_ARG


def test_binding_struct_layouts_match_the_header(tmp_path):
    # the header is plain C: compile a probe against it and compare sizes and member offsets with the ctypes mirrors
    import subprocess
    from paper_2407_17029_b200 import binding
    members = {"qblora_qweight": ["d_in", "d_out", "block_in", "block_out", "qfmt", "code", "codes", "alpha", "beta", "code_bits"],
               "qblora_adapter": ["lambda_in", "lambda_out", "rank", "scaling", "A", "B", "scale_op"]}
    lines = ['#include <stdio.h>', '#include <stddef.h>', '#include "qblora.h"', 'int main(void) {']
    for s, ms in members.items():
        lines.append(f'  printf("{s} %zu\\n", sizeof({s}));')
        for m in ms:
            lines.append(f'  printf("{s}.{m} %zu\\n", offsetof({s}, {m}));')
    lines += ['  printf("enum %d %d %d\\n", QBLORA_SCALE_AVGPOOL_REPEAT, QBLORA_SCALE_TRUNCATE_ZEROPAD, QBLORA_SCALE_SAMPLE_ZEROFILL);',
              '  return 0;', '}']
    src = tmp_path / "probe.c"
    src.write_text("\n".join(lines))
    exe = tmp_path / "probe"
    subprocess.run(["gcc", "-std=c99", "-I", os.path.join(ROOT, "include"), str(src), "-o", str(exe)], check=True)
    out = dict(l.split(" ", 1) for l in subprocess.run([str(exe)], check=True, capture_output=True, text=True).stdout.splitlines())
    mirrors = {"qblora_qweight": binding._CQWeight, "qblora_adapter": binding._CAdapter}
    for s, ms in members.items():
        assert int(out[s]) == ctypes.sizeof(mirrors[s])
        assert [f[0] for f in mirrors[s]._fields_] == ms
        for m in ms:
            assert int(out[f"{s}.{m}"]) == getattr(mirrors[s], m).offset, (s, m)
    assert out["enum"].split() == [str(binding.SCALE_AVGPOOL_REPEAT), str(binding.SCALE_TRUNCATE_ZEROPAD),
                                   str(binding.SCALE_SAMPLE_ZEROFILL)]
