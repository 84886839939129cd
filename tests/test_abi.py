"""Host-side checks that need no GPU: the library builds, loads and exports what the header declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2606_12243_b200 import build
    path = build.build()
    return ctypes.CDLL(path)


def _declared():
    text = open(os.path.join(ROOT, "include", "viasd.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(viasd_[a-z_0-9]+)\s*\(", text)))


def test_header_symbols_are_exported(lib):
    names = _declared()
    assert {"viasd_init_model", "viasd_verify_step", "viasd_slim_forward", "viasd_full_forward",
            "viasd_tier_accept", "viasd_kv_commit"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n


def test_binding_lists_every_export():
    from paper_2606_12243_b200 import binding
    assert sorted(binding.EXPORTS) == _declared()


def test_host_only_calls(lib):
    from paper_2606_12243_b200 import binding as vb
    assert vb.lib().viasd_strerror(0) == b"ok"
    assert vb.lib().viasd_strerror(vb.VIASD_EINVAL) == b"invalid argument"
    cfg = vb.make_config(32, 4096, 32, 32, 128, 11008, 32000, "bf16", 1, 1033, 9)
    n = vb.workspace_bytes(cfg, 16)
    assert 1 << 20 < n < 1 << 30
    bad = vb.make_config(32, 4096, 32, 5, 128, 11008, 32000, "bf16", 1, 1033, 9)   # heads % kv_heads != 0
    assert vb.workspace_bytes(bad, 16) == 0
    assert vb.workspace_bytes(vb.make_config(32, 4096, 32, 32, 128, 11008, 32000, "bf16", 1, 1033, 65), 16) == 0


def test_struct_layouts_match_header():
    """Sizes the C compiler gives the public structs equal the ctypes mirrors."""
    import subprocess, tempfile, textwrap
    from paper_2606_12243_b200 import binding as vb
    src = textwrap.dedent('''
        #include <stdio.h>
        #include "viasd.h"
        int main(void) {
            printf("%zu %zu %zu %zu %zu %zu %zu\\n", sizeof(viasd_config), sizeof(viasd_weights), sizeof(viasd_cache),
                   sizeof(viasd_draft), sizeof(viasd_params), sizeof(viasd_result), sizeof(viasd_stats));
            return 0;
        }''')
    with tempfile.TemporaryDirectory() as d:
        c = os.path.join(d, "t.c")
        open(c, "w").write(src)
        exe = os.path.join(d, "t")
        subprocess.check_call(["gcc", "-I", os.path.join(ROOT, "include"), c, "-o", exe])
        sizes = [int(x) for x in subprocess.check_output([exe]).split()]
    mirrors = [vb.Config, vb.Weights, vb.Cache, vb.Draft, vb.Params, vb.Result, vb.Stats]
    assert sizes == [ctypes.sizeof(m) for m in mirrors]
