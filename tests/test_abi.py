"""The C-ABI library builds, loads and exports every function the header declares (no GPU needed)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "inferturbo.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(it_[a-z_]+)\s*\(", text)))


def test_header_declares_the_boundary_calls():
    names = declared_functions()
    for required in ("it_graph_create", "it_split_hubs", "it_layer_forward", "it_infer"):
        assert required in names


def test_library_exports_every_declared_symbol():
    from paper_2307_00228_b200 import build
    lib = ctypes.CDLL(build.build())
    for name in declared_functions():
        assert hasattr(lib, name), name


def test_binding_has_the_same_names_and_fails_loudly_without_the_library(monkeypatch):
    import paper_2307_00228_b200 as pkg
    from paper_2307_00228_b200 import binding
    for name in declared_functions():
        assert hasattr(pkg, name) or hasattr(binding, name), name
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", "/nonexistent/libinferturbo.so")
    with pytest.raises(ImportError):
        binding.lib()


def test_status_strings():
    from paper_2307_00228_b200 import binding
    assert [binding.it_status_string(i) for i in range(8)] == binding.STATUS_NAMES


def test_layer_desc_struct_matches_the_header_layout():
    """Field order and sizes of the ctypes mirror follow the typedef in the header."""
    from paper_2307_00228_b200 import binding
    text = open(os.path.join(ROOT, "include", "inferturbo.h")).read()
    body = re.search(r"typedef struct \{(.*?)\} it_layer_desc;", text, flags=re.S).group(1)
    body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
    names = []
    for decl in body.split(";"):
        decl = decl.strip()
        if not decl:
            continue
        parts = decl.replace("*", " ").split()
        names += [p.strip(",") for p in parts[1:] if p.strip(",") not in ("void", "float", "const")]
    assert names == [f[0] for f in binding.it_layer_desc._fields_]
    # sizes and offsets as the C compiler sees them
    import subprocess
    import tempfile
    fields = [f[0] for f in binding.it_layer_desc._fields_]
    prog = "#include <stdio.h>\n#include <stddef.h>\n#include \"inferturbo.h\"\nint main(void){printf(\"%zu\", sizeof(it_layer_desc));" + \
        "".join(f'printf(" %zu", offsetof(it_layer_desc, {f}));' for f in fields) + "return 0;}\n"
    with tempfile.TemporaryDirectory() as d:
        src, exe = os.path.join(d, "t.c"), os.path.join(d, "t")
        open(src, "w").write(prog)
        subprocess.check_call(["gcc", "-I", os.path.join(ROOT, "include"), src, "-o", exe])
        nums = [int(t) for t in subprocess.check_output([exe]).split()]
    assert nums[0] == ctypes.sizeof(binding.it_layer_desc)
    assert nums[1:] == [getattr(binding.it_layer_desc, f).offset for f in fields]
