"""Host-side checks that need no GPU: the library builds, loads and exports every symbol the header
declares; host helpers agree with the literal tables; multi-process sharding logic on gloo."""
import ctypes
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2109_10060_b200.build import build
    build()
    import paper_2109_10060_b200 as dsn
    return dsn


def test_library_exports_every_declared_symbol(lib):
    header = open(os.path.join(ROOT, "include", "dsn.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = sorted(set(re.findall(r"\b(dsn_[a-z_0-9]+)\s*\(", header)))
    assert "dsn_gate" in declared and "dsn_route" in declared and "dsn_sliced_linear" in declared
    assert "dsn_sliced_conv" in declared and "dsn_layer_forward" in declared
    handle = lib.load_library()
    for name in declared:
        assert hasattr(handle, name), f"{name} declared in dsn.h but not exported"
    assert sorted(lib.EXPORTS) == declared


def test_struct_layouts_match_header_sizes(lib, tmp_path):
    """sizeof of every descriptor as the C compiler lays it out equals the ctypes mirror."""
    import subprocess
    names = {"dsn_routing": lib.Routing, "dsn_gate_desc": lib.GateDesc, "dsn_linear_desc": lib.LinearDesc,
             "dsn_conv_desc": lib.ConvDesc, "dsn_layer_desc": lib.LayerDesc,
             "dsn_attention_desc": lib.AttentionDesc, "dsn_depthwise_desc": lib.DepthwiseDesc, "dsn_stats": lib.Stats}
    src = tmp_path / "sizes.c"
    body = "".join(f'printf("{n} %zu\\n", sizeof({n}));' for n in names)
    src.write_text('#include <stdio.h>\n#include "dsn.h"\nint main(void){' + body + "return 0;}\n")
    exe = tmp_path / "sizes"
    subprocess.run(["gcc", "-std=c99", "-I", os.path.join(ROOT, "include"), str(src), "-o", str(exe)], check=True)
    out = subprocess.run([str(exe)], check=True, capture_output=True, text=True).stdout.split()
    got = dict(zip(out[0::2], map(int, out[1::2])))
    for n, cls in names.items():
        assert got[n] == ctypes.sizeof(cls), n


def test_widths_helper_matches_tables(lib):
    from dsn_workloads import RATIOS_14, WIDTHS_14
    for C in (64, 128, 256, 512, 640):
        assert lib.dsn_widths_from_ratios(C, RATIOS_14) == WIDTHS_14[C]
    assert lib.dsn_widths_from_ratios(256, [0.25, 0.5, 0.75, 1.0]) == [64, 128, 192, 256]
    with pytest.raises(lib.DsnError):
        lib.dsn_widths_from_ratios(256, [0.0])


def test_executed_macs_counter(lib):
    from oracle import dsn_oracle as O
    idx = np.array([0, 2, 2, 1, 0, 2])
    k_in, k_out = [4, 8, 16], [3, 6, 9]
    counts = np.bincount(idx, minlength=3).tolist()
    assert lib.dsn_executed_macs(counts, 7, k_in, k_out, 3) == O.executed_macs(idx, 7, k_in, k_out, K=3)


def test_strerror_and_no_device_is_an_error_not_a_crash(lib):
    assert lib.dsn_strerror(0) == "ok"
    assert "index" in lib.dsn_strerror(lib.ERR_BAD_INDEX)
    import torch
    if not torch.cuda.is_available():
        with pytest.raises(lib.DsnError):
            lib.Context(0)


def test_package_has_no_cpu_fallback():
    """The product path may not reach the oracle or any CPU implementation."""
    pkg = os.path.join(ROOT, "paper_2109_10060_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text.replace("no CPU or framework fallback", ""), f
