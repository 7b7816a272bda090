"""The C-ABI library loads without a GPU and exports every symbol that
include/falcon.h declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    names = set()
    inc = os.path.join(ROOT, "include")
    for f in os.listdir(inc):
        if f.endswith(".h"):
            text = open(os.path.join(inc, f)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\b(falcon_[a-z_0-9]+)\s*\(", text))
    return sorted(names)


@pytest.fixture(scope="module")
def lib():
    from paper_2412_12639_b200 import build
    return ctypes.CDLL(build.build())


def test_header_declares_the_three_calls():
    names = declared_functions()
    for n in ("falcon_tree_attn", "falcon_tree_accept", "falcon_kv_compact", "falcon_create", "falcon_destroy"):
        assert n in names


def test_library_exports_every_declared_symbol(lib):
    for n in declared_functions():
        assert hasattr(lib, n), n


def test_host_only_entry_points(lib):
    from paper_2412_12639_b200 import binding
    assert binding.falcon_tree_validate_host([-1, 0, 0, 1]) == binding.OK
    assert binding.falcon_tree_validate_host([-1, 2, 0]) == binding.ERR_BAD_TREE
    assert binding.falcon_tree_validate_host([0]) == binding.ERR_BAD_TREE
    assert binding.falcon_tree_validate_host([-1] + [0] * 128) == binding.ERR_UNSUPPORTED
    assert binding.status_string(0) == "ok"
    assert "tree" in binding.status_string(binding.ERR_BAD_TREE)


def test_binding_structs_match_header_field_order():
    # the ctypes structures list the fields of the C structs in declaration order
    from paper_2412_12639_b200 import binding
    text = open(os.path.join(ROOT, "include", "falcon.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    for cname, struct in (("falcon_tree_desc", binding.TreeDesc), ("falcon_attn_args", binding.AttnArgs),
                          ("falcon_accept_args", binding.AcceptArgs), ("falcon_compact_args", binding.CompactArgs),
                          ("falcon_gather_args", binding.GatherArgs),
                          ("falcon_lm_argmax_args", binding.LmArgmaxArgs)):
        end = re.search(r"\}\s*%s;" % cname, text).start()
        body = text[text.rfind("typedef struct {", 0, end) + len("typedef struct {"):end]
        fields = []
        for decl in body.split(";"):
            decl = decl.strip()
            if not decl:
                continue
            for part in decl.split(","):
                fields.append(re.findall(r"([A-Za-z_0-9]+)\s*$", part.strip())[0])
        assert fields == [f[0] for f in struct._fields_], cname


def test_binding_structs_match_the_compiled_layout(tmp_path):
    """The header compiles as plain C, and the size of every argument struct and the offset of every
    field, as the C compiler lays them out, equal those of the ctypes structures."""
    import shutil
    import subprocess
    from paper_2412_12639_b200 import binding
    cc = shutil.which("gcc") or shutil.which("cc")
    if cc is None:
        pytest.skip("no C compiler")
    structs = (("falcon_tree_desc", binding.TreeDesc), ("falcon_attn_args", binding.AttnArgs),
               ("falcon_accept_args", binding.AcceptArgs), ("falcon_topm_args", binding.TopmArgs),
               ("falcon_compact_args", binding.CompactArgs), ("falcon_gather_args", binding.GatherArgs),
               ("falcon_lm_argmax_args", binding.LmArgmaxArgs))
    lines = ['#include <stdio.h>', '#include <stddef.h>', '#include "falcon.h"', 'int main(void) {']
    for cname, st in structs:
        lines.append('  printf("%s %%zu\\n", sizeof(%s));' % (cname, cname))
        for fname, _ in st._fields_:
            lines.append('  printf("%s.%s %%zu\\n", offsetof(%s, %s));' % (cname, fname, cname, fname))
    lines += ['  return 0;', '}']
    src = tmp_path / "layout.c"
    src.write_text("\n".join(lines))
    exe = tmp_path / "layout"
    subprocess.run([cc, "-std=c99", "-Wall", "-Werror", "-I", os.path.join(ROOT, "include"), str(src), "-o", str(exe)],
                   check=True)
    got = dict(line.split() for line in subprocess.run([str(exe)], check=True, capture_output=True,
                                                       text=True).stdout.splitlines())
    for cname, st in structs:
        assert int(got[cname]) == ctypes.sizeof(st), cname
        for fname, _ in st._fields_:
            assert int(got["%s.%s" % (cname, fname)]) == getattr(st, fname).offset, "%s.%s" % (cname, fname)
