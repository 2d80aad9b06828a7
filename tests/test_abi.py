"""The C-ABI library builds, loads, and exports every symbol its header declares (no GPU)."""
import ctypes
import os
import re

import pytest
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    names = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\b(sb_[a-z0-9_]+)\s*\(", text))
    return names


def test_library_builds_and_exports_every_declared_symbol():
    from paper_2602_17698_b200 import build, binding
    path = build.build()
    assert os.path.exists(path)
    lib = ctypes.CDLL(path)
    declared = _declared()
    assert {"sb_calib_moments", "sb_reorder_channels", "sb_block_scores", "sb_allocate_bits",
            "sb_pack_blocks"} <= declared
    for name in declared:
        assert hasattr(lib, name), f"{name} declared in include/ but not exported"
    assert set(binding.EXPORTS) <= declared


def test_every_export_has_its_argument_types_declared():
    """Without argtypes ctypes passes Python ints as 32-bit C ints: the upper half of a 64-bit
    parameter on the stack would be whatever was there."""
    from paper_2602_17698_b200 import binding
    lib = binding.lib()
    header = open(os.path.join(ROOT, "include", "scalebits.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    for name in binding.EXPORTS:
        fn = getattr(lib, name)
        assert fn.argtypes is not None, name
        m = re.search(r"\b" + name + r"\s*\(([^;]*?)\)\s*;", header, flags=re.S)
        assert m, name
        n_params = len([p for p in m.group(1).split(",") if p.strip() and p.strip() != "void"])
        assert len(fn.argtypes) == n_params, (name, len(fn.argtypes), n_params)


def test_binding_has_a_method_per_entry_point():
    from paper_2602_17698_b200 import binding
    for name in _declared():
        short = name[3:]
        if short in ("create", "destroy", "last_error"):
            continue
        assert hasattr(binding.Context, short) or hasattr(binding, short), short


@pytest.mark.skipif(torch.cuda.is_available(), reason="checks the no-GPU failure mode")
def test_no_cpu_fallback():
    """Without a CUDA device the product path fails loudly instead of computing on the CPU."""
    from paper_2602_17698_b200 import binding
    with pytest.raises(RuntimeError):
        binding.Context()
    h = ctypes.c_void_p()
    assert binding.lib().sb_create(ctypes.byref(h), 0, None) == binding.SB_ERR_CUDA
    assert not h.value


def test_product_code_never_imports_the_oracle():
    pkg = os.path.join(ROOT, "paper_2602_17698_b200")
    for dirpath, _, files in os.walk(pkg):
        for fn in files:
            if fn.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, fn)).read()
                assert not re.search(r"^\s*(from|import)\s+oracle\b", text, flags=re.M), fn
                assert "libsbo" not in text and "scalebits_oracle" not in text, fn


def test_report_structs_of_the_binding_match_the_header(tmp_path):
    """The two report structs are laid out by a C compiler from the header and by ctypes from the
    binding's field lists: same size and same offset for every field, and a report decoded from
    raw bytes (as `read_report` does for the device copy) returns the values that were stored."""
    import subprocess
    from paper_2602_17698_b200 import binding
    src = tmp_path / "layout.c"
    fields = {"sb_alloc_report": [f for f, _ in binding.AllocReport._fields_],
              "sb_step_report": [f for f, _ in binding.StepReport._fields_]}
    lines = ['#include <stddef.h>', '#include <stdio.h>', '#include "scalebits.h"', "int main(void) {"]
    for struct, names in fields.items():
        lines.append(f'  printf("{struct} %zu", sizeof({struct}));')
        for f in names:
            lines.append(f'  printf(" %zu", offsetof({struct}, {f}));')
        lines.append('  printf("\\n");')
    lines += ["  return 0;", "}"]
    src.write_text("\n".join(lines))
    exe = tmp_path / "layout"
    subprocess.run(["gcc", "-I", os.path.join(ROOT, "include"), "-o", str(exe), str(src)], check=True)
    out = subprocess.run([str(exe)], check=True, capture_output=True, text=True).stdout.split("\n")
    for line, (struct, names), cls in zip(out, fields.items(), (binding.AllocReport, binding.StepReport)):
        got = line.split()
        assert got[0] == struct and int(got[1]) == ctypes.sizeof(cls), line
        assert [int(x) for x in got[2:]] == [getattr(cls, f).offset for f in names], line
    rep = binding.AllocReport(cap_bits=1 << 40, used_bits=(1 << 40) - 5, iterations=13, accepted=1, rejected=2,
                              expansions=10, proxy_loss_init=2.5, proxy_loss_final=0.125)
    for i in range(8):
        rep.level_hist[i] = 100 + i
    raw = torch.frombuffer(bytearray(bytes(rep)) + bytearray(16), dtype=torch.uint8)   # a larger buffer, as the workspace's
    assert binding.Context.read_report(raw) == rep.as_dict()
