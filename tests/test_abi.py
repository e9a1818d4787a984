"""The C-ABI library loads and exports every symbol include/dspark.h declares (no GPU needed)."""
import os
import re

import pytest

from paper_2607_05147_b200 import binding as B
from paper_2607_05147_b200 import build as build_mod

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    src = open(os.path.join(ROOT, "include", "dspark.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(dspark_[a-z_0-9]+)\s*\(", src)))


def test_header_symbols_are_exported():
    build_mod.build()
    L = B.lib()
    names = _declared()
    assert len(names) >= 15
    for n in names:
        assert hasattr(L, n), f"{n} declared in dspark.h but not exported"
    assert set(B.EXPORTS) == set(names)


def test_host_only_entry_points():
    L = B.lib()
    assert L.dspark_version() >= 100
    assert L.dspark_status_string(4).decode() == "workspace too small"
    assert L.dspark_kernel_name(B.K_STREAM).decode() == "stream_stats"
    # workspace queries are pure host arithmetic
    assert B.dspark_verify_workspace_bytes(64, 352, 129280) > 2 * 352 * 127 * 8
    assert B.dspark_verify_workspace_bytes(0, 1, 10) == 0
    assert B.dspark_schedule_workspace_bytes(512, 32) >= 16384 * (4 + 8 + 8 + 4)
    assert B.dspark_schedule_workspace_bytes(1 << 20, 2) == 0          # beyond the supported size


def test_uniforms_match_oracle_bit_for_bit():
    import oracle
    for seed in (0, 1, 0xDEADBEEFCAFEF00D):
        for r in (0, 1, 77, 1023, 65537):
            for j in (0, 1, 5, 31):
                assert B.dspark_uniforms(seed, r, j) == oracle.uniforms(seed, r, j)


def test_uniforms_match_oracle_on_a_million_counters():
    # two independent Philox4x32-10 implementations (the library's and the oracle's), 10^6 (seed, request, position)
    # counters: low and high key words, requests and positions across several powers of two
    import ctypes as C
    import numpy as np
    import oracle
    L, O = B.lib(), oracle.lib()
    rng = np.random.default_rng(123)
    seeds = [0, 1, 0xFFFFFFFF, 0x100000000, 0xDEADBEEFCAFEF00D] + [int(x) for x in rng.integers(0, 2**63, size=95, dtype=np.uint64)]
    reqs = [0, 1, 2, 255, 256, 65535, 65536, 2**31 - 1, 2**32 - 1] + [int(x) for x in rng.integers(0, 2**32, size=91, dtype=np.uint64)]
    poss = [0, 1, 2, 3, 31, 32, 4095, 2**32 - 1] + [int(x) for x in rng.integers(0, 2**20, size=92, dtype=np.uint64)]
    a, b, c, d = C.c_float(), C.c_float(), C.c_float(), C.c_float()
    n = 0
    for seed in seeds:
        s64 = C.c_uint64(seed)
        for r in reqs:
            r32 = C.c_uint32(r)
            for j in poss:
                j32 = C.c_uint32(j)
                L.dspark_uniforms(s64, r32, j32, C.byref(a), C.byref(b))
                O.orc_uniforms(s64, r32, j32, C.byref(c), C.byref(d))
                assert a.value == c.value and b.value == d.value, (seed, r, j)
                assert 0.0 <= a.value < 1.0 and 0.0 <= b.value < 1.0
                n += 1
    assert n == 10**6


def test_cpu_tensors_are_refused():
    import torch
    with pytest.raises(B.DsparkError):
        B.dspark_build_offsets(torch.zeros(4, dtype=torch.int32), torch.zeros(5, dtype=torch.int32))
