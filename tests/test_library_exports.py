"""CPU checks of the boundary: the C-ABI library builds, loads and exports every symbol that
include/ffint8.h declares (no compute calls: there is no GPU here)."""
import os
import re

from paper_2506_22771_b200 import binding as ffb

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "ffint8.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ff_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = ffb.load()
    names = _declared()
    assert len(names) >= 13
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(ffb.EXPORTS) == names


def test_struct_layouts_match_header_field_order():
    text = open(os.path.join(ROOT, "include", "ffint8.h")).read()
    body = re.search(r"typedef struct \{([^}]*)\} ff_layer_bufs;", text, flags=re.S).group(1)
    body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
    fields = re.findall(r"(?:\*\s*|int32_t\s+)([A-Za-z_]+)\s*;", body)      # the pointers, then the INT32 row pitches
    assert fields == [f[0] for f in ffb.ff_layer_bufs._fields_]
    body = re.search(r"typedef struct \{([^}]*)\} ff_layer_desc;", text, flags=re.S).group(1)
    body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
    names = []
    for decl in body.split(";"):
        decl = decl.strip()
        if decl:
            names += [n.strip() for n in decl.split(None, 1)[1].split(",")]
    assert names == [f[0] for f in ffb.ff_layer_desc._fields_]


def test_create_without_gpu_fails_cleanly():
    import torch
    if torch.cuda.is_available():
        return
    try:
        ffb.ff_create(0)
    except ffb.FFError as e:
        assert e.code in (ffb.FF_ERR_CUDA, ffb.FF_ERR_UNSUPPORTED_ARCH)
    else:
        raise AssertionError("ff_create must fail when there is no CUDA device")
