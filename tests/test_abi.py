"""Host-side checks that need no GPU: the library builds, loads, and exports what the header declares."""
import os
import re

from paper_2412_11272_b200 import build as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "wf_encoder.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(wf_[a-z0-9_]+)\s*\(", text)))


def test_library_builds_and_exports_every_declared_symbol():
    B.build()
    from paper_2412_11272_b200 import binding
    lib = binding.load_library()
    names = _declared()
    assert "wf_encode" in names and "wf_logmel" in names and "wf_encoder_create" in names
    for name in names:
        assert hasattr(lib, name), name
    assert set(binding.EXPORTS) <= set(names)


def test_binding_structs_match_header_field_order():
    from paper_2412_11272_b200 import binding
    text = open(os.path.join(ROOT, "include", "wf_encoder.h")).read()
    cfg = re.search(r"typedef struct \{(.*?)\} wf_config;", text, flags=re.S).group(1)
    cfg = re.sub(r"/\*.*?\*/", "", cfg, flags=re.S)
    fields = [f.strip() for decl in cfg.split(";") for f in re.sub(r"^\s*(int|long)\s+", "", decl.strip()).split(",") if f.strip()]
    assert fields == [n for n, _ in binding.wf_config._fields_]
    w = re.search(r"typedef struct \{(.*?)\} wf_weights;", text, flags=re.S).group(1)
    w = re.sub(r"/\*.*?\*/", "", w, flags=re.S)
    names = re.findall(r"\*\s*(?:const\s*\*\s*)?([a-z0-9_]+)\s*[,;]", w)
    assert names == [n for n, _ in binding.wf_weights._fields_]
