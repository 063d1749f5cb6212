"""The binding's ctypes structures against the C header: a small C program compiled with gcc prints the size of
every struct in include/wpp.h and the offset of every field; the ctypes mirror must agree field by field."""
import ctypes
import os
import re
import subprocess

import paper_2609_35263_b200.binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
PAIRS = {"wpp_batch_desc": B.BatchDesc, "wpp_plan_opts": B.PlanOpts, "wpp_plan_info": B.PlanInfo,
         "wpp_wave_config": B.WaveConfig, "wpp_wave_state": B.WaveState, "wpp_wave_info": B.WaveInfo,
         "wpp_kda_desc": B.KdaDesc}


def _c_fields(name, hdr):
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    body = re.search(r"typedef struct \{([^{}]*)\}\s*%s;" % name, hdr).group(1)
    fields = []
    for decl in body.split(";"):
        decl = decl.strip()
        if decl:
            names = decl.split(None, 1)[1]
            fields += [n.strip() for n in names.split(",")]
    return fields


def test_ctypes_structures_match_the_header(tmp_path):
    hdr = open(os.path.join(ROOT, "include", "wpp.h")).read()
    lines = ['#include <stdio.h>', '#include <stddef.h>', '#include "wpp.h"', "int main(void) {"]
    for cname in PAIRS:
        lines.append(f'printf("{cname} size %zu\\n", sizeof({cname}));')
        for f in _c_fields(cname, hdr):
            lines.append(f'printf("{cname} {f} %zu\\n", offsetof({cname}, {f}));')
    lines += ["return 0;", "}"]
    src, exe = tmp_path / "abi.c", tmp_path / "abi"
    src.write_text("\n".join(lines))
    subprocess.check_call(["gcc", "-I", os.path.join(ROOT, "include"), str(src), "-o", str(exe)])
    seen = {}
    for line in subprocess.check_output([str(exe)], text=True).splitlines():
        cname, field, value = line.split()
        seen.setdefault(cname, {})[field] = int(value)
    for cname, cls in PAIRS.items():
        got = {"size": ctypes.sizeof(cls)}
        got.update({n: getattr(cls, n).offset for n, _ in cls._fields_})
        assert got == seen[cname], cname


def test_entry_points_reject_a_null_context_without_touching_a_gpu():
    """Every device entry point validates its arguments on the host first: with no context nothing is launched."""
    lib = B.load_library()
    desc = B.KdaDesc(1, 1, 128, 128, 1, 0, 0, 0, 4)
    assert lib.wpp_kda_chunk(None, ctypes.byref(desc), *([None] * 13), 0, None, None) == 1          # WPP_ERR_INVALID_ARG
    assert lib.wpp_hash_blocks(None, None, None, None, 1, 16, 0, None, None, 1, None) == 1
    bd = B.make_desc(1, 2, 1, 128, 16, 4, 8)
    assert lib.wpp_kv_append(None, ctypes.byref(bd), *([None] * 11)) == 1
