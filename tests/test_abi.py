"""Host-only checks of the C-ABI library: it builds, loads, and exports every symbol include/a3.h declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib_path():
    from paper_2511_17560_b200 import build
    return build.build()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "a3.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(a3_[a-z0-9_]+)\s*\(", text)))


def test_header_symbols_are_exported(lib_path):
    lib = ctypes.CDLL(lib_path)
    syms = declared_symbols()
    assert {"a3_rope_rerotate", "a3_query_scores", "a3_topk_select", "a3_recompute_layer", "a3_scatter_kv",
            "a3_fuse_request"} <= set(syms)
    for s in syms:
        assert hasattr(lib, s), s


def test_binding_lists_the_same_symbols(lib_path):
    from paper_2511_17560_b200 import a3
    assert sorted(a3.EXPORTS) == declared_symbols()
    a3._load()


def test_no_undeclared_a3_symbols_are_exported(lib_path):
    """Everything the library exports under the a3_ prefix is declared (and documented) in include/a3.h."""
    import subprocess
    out = subprocess.run(["nm", "-D", "--defined-only", lib_path], check=True, capture_output=True, text=True).stdout
    exported = sorted({ln.split()[-1] for ln in out.splitlines() if ln.split() and ln.split()[-1].startswith("a3_")})
    assert exported == declared_symbols()


def test_host_only_entry_points(lib_path):
    from paper_2511_17560_b200 import a3
    lib = a3._load()
    assert a3.recompute_count(0.15, 5152, 5120) == 772
    assert a3.recompute_count(0.15, 528, 512) == 79
    assert a3.recompute_count(1.0, 528, 512) == 512
    assert a3.recompute_count(0.0, 528, 512) == 0
    assert a3.recompute_count(0.3, 10, 10) == 3
    assert lib.a3_status_string(0) == b"ok"
    assert lib.a3_status_string(-3) == b"workspace too small"
    # argument validation happens before any CUDA call
    assert lib.a3_create(None, None, None) == -1
    assert lib.a3_fuse_request(None, None, None, 0, None) == -1
    assert lib.a3_rope_rerotate(None, None, 0, 0, None, None, 0, 0, 0, 0, None) == -1
    assert lib.a3_set_option(None, 0, 0) == -1
    assert lib.a3_scores_workspace_bytes(None, 10) == 0
    assert lib.a3_swiglu_rows(None, 0, None, None, 0, None) == -1
    assert lib.a3_topk_select(None, None, 0, 0, 0, None, None) == -1
    assert lib.a3_layer_workspace_bytes(None, 10) == 0


def test_struct_layouts_match_header(tmp_path):
    """sizeof/offsetof as the C compiler sees include/a3.h against the ctypes mirrors of the binding."""
    import subprocess
    from paper_2511_17560_b200 import a3
    structs = {"a3_chunk_ref": a3.ChunkRef, "a3_layer_weights": a3.LayerWeights, "a3_request": a3.Request,
               "a3_model_desc": a3.ModelDesc, "a3_host_io": a3.HostIO, "a3_profile_entry": a3.ProfileEntry}
    lines = []
    for cname, cls in structs.items():
        lines.append(f'printf("{cname} size %zu\\n", sizeof({cname}));')
        for fname, _ in cls._fields_:
            lines.append(f'printf("{cname} {fname} %zu\\n", offsetof({cname}, {fname}));')
    src = tmp_path / "layout.c"
    src.write_text('#include <stdio.h>\n#include <stddef.h>\n#include "a3.h"\nint main(void) {\n' + "\n".join(lines) + "\nreturn 0; }\n")
    exe = tmp_path / "layout"
    inc = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "include")
    subprocess.run(["gcc", "-std=c99", "-I", inc, str(src), "-o", str(exe)], check=True)
    got = {}
    for ln in subprocess.run([str(exe)], check=True, capture_output=True, text=True).stdout.splitlines():
        cname, field, val = ln.split()
        got[(cname, field)] = int(val)
    for cname, cls in structs.items():
        assert ctypes.sizeof(cls) == got[(cname, "size")], cname
        for fname, _ in cls._fields_:
            assert getattr(cls, fname).offset == got[(cname, fname)], (cname, fname)
    assert ctypes.sizeof(a3.ChunkRef) == 40


def test_host_only_helpers_match_oracle():
    """a3_chunk_edge_rows, a3_recompute_count and a3_evict_count are host arithmetic: no GPU needed."""
    import numpy as np
    from oracle import a3_oracle as O
    from paper_2511_17560_b200 import a3
    rng = np.random.default_rng(0)
    for _ in range(50):
        lens = rng.integers(0, 90, size=rng.integers(1, 9)).tolist()
        m = int(rng.integers(1, 30))
        ns = int(rng.integers(0, max(1, lens[0] + 1)))
        assert a3.chunk_edge_rows(lens, m, ns).tolist() == O.chunk_edge_rows(lens, m, ns).tolist()
    assert a3.chunk_edge_rows((512,) * 10, 20).size == 400
    for ratio, n, nc in ((0.15, 5152, 5120), (1.0, 100, 90), (0.0, 10, 10), (0.3, 10, 2), (0.15, 20, 20)):
        assert a3.recompute_count(ratio, n, nc) == O.recompute_count(ratio, n, nc)
    assert a3.evict_count(1024, 40, 5120, 32) == 952 and a3.evict_count(10, 40, 5120, 32) == 0 and a3.evict_count(10**6, 0, 100, 5) == 100
