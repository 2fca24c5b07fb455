"""Host-side checks of the C ABI that need no GPU: the library loads, exports every declared symbol,
sizes its workspace sanely and rejects bad arguments before launching anything."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def fq():
    from paper_2510_24061_b200 import build
    build.build()
    from paper_2510_24061_b200 import binding
    return binding


def test_library_exports_every_declared_symbol(fq):
    header = open(os.path.join(ROOT, "include", "falqon.h")).read()
    declared = set(re.findall(r"\b(falqon_[a-z_]+)\s*\(", header))
    assert declared == set(fq.EXPORTS)
    for name in declared:
        assert hasattr(fq.lib, name), name


def test_chain_header_symbols_are_exported(fq):
    header = open(os.path.join(ROOT, "include", "falqon_chain.h")).read()
    declared = set(re.findall(r"\b(falqon_chain_[a-z_]+)\s*\(", header))
    from paper_2510_24061_b200 import stack
    assert declared == set(stack.CHAIN_EXPORTS)
    for name in declared:
        assert hasattr(fq.lib, name), name
    fake = 0x10000
    assert fq.lib.falqon_chain_combine(fake, None, C.c_float(1), None, C.c_float(1), None, C.c_float(1), None, C.c_float(1),
                                       64, None, None) == fq.ERR_INVALID_ARG
    assert stack.lib.falqon_chain_rmsnorm(fake, fake, fake, 4, 12, C.c_float(1e-6), None, None) == fq.ERR_INVALID_ARG   # cols % 8


def test_workspace_layout(fq):
    m, n, r, T = 4096, 4096, 64, 4096
    total = fq.workspace_bytes(m, n, r, T)
    assert total >= T * max(m, n) + T * r
    seen = []
    for which in (fq.WS_XQ, fq.WS_OAQ_T, fq.WS_SCALES, fq.WS_SCORE):
        off, size = fq.workspace_region(m, n, r, T, which)
        assert off % 256 == 0 and off + size <= total
        seen.append((off, off + size))
    seen.sort()
    assert all(a[1] <= b[0] for a, b in zip(seen, seen[1:]))          # regions do not overlap
    # score region does not move with T, so a proxy update finds it in a workspace sized for any T
    assert fq.workspace_region(m, n, r, 1, fq.WS_SCORE) == fq.workspace_region(m, n, r, T, fq.WS_SCORE)
    for bad in [(4096, 4100, 64, 16), (4096, 4096, 12, 16), (4096, 4096, 512, 16), (8, 4096, 64, 16), (4096, 4096, 64, 0)]:
        assert fq.workspace_bytes(*bad) == 0


def test_bad_arguments_are_rejected_on_the_host(fq):
    lib = fq.lib
    fake = 0x10000  # an aligned non-null address that is never dereferenced on these paths
    layer = fq.falqon_layer(256, 256, 16, fake, fake, fake, 0, 0)
    big = 1 << 40
    inv, wsp = fq.ERR_INVALID_ARG, fq.ERR_WORKSPACE
    # quantize
    assert lib.falqon_quantize(None, 0, 4, 16, 0, 0, None, 1.0, fake, fake, None, fake, 8192, None) == inv
    assert lib.falqon_quantize(fake, 0, 4, 20, 0, 0, None, 1.0, fake, fake, None, fake, 8192, None) == inv   # cols % 16
    assert lib.falqon_quantize(fake, 0, 4, 16, 7, 0, None, 1.0, fake, fake, None, fake, 8192, None) == inv   # format
    assert lib.falqon_quantize(fake + 4, 0, 4, 16, 0, 0, None, 1.0, fake, fake, None, fake, 8192, None) == inv  # alignment
    assert lib.falqon_quantize(fake, 0, 4, 16, 0, 0, None, 1.0, fake, None, None, fake, 8192, None) == inv   # nowhere to put the scale
    assert lib.falqon_quantize(fake, 0, 4, 16, 0, 0, None, 1.0, fake, fake, None, None, 0, None) == wsp
    # forward
    assert lib.falqon_melded_forward(None, fake, 0, 16, fake, 0, fake, fake, None, fake, big, None) == inv
    assert lib.falqon_melded_forward(C.byref(layer), None, 0, 16, fake, 0, fake, fake, None, fake, big, None) == inv
    assert lib.falqon_melded_forward(C.byref(layer), fake, 0, 0, fake, 0, fake, fake, None, fake, big, None) == inv
    assert lib.falqon_melded_forward(C.byref(layer), fake, 3, 16, fake, 0, fake, fake, None, fake, big, None) == inv
    assert lib.falqon_melded_forward(C.byref(layer), fake, 0, 16, fake, 0, fake, fake, None, fake, 1024, None) == wsp
    bad_flags = fq.falqon_layer(256, 256, 16, fake, fake, fake, 0, 8)     # an undefined flag bit
    assert lib.falqon_melded_forward(C.byref(bad_flags), fake, 0, 16, fake, 0, fake, fake, None, fake, big, None) == inv
    fused = fq.falqon_layer(256, 256, 16, fake, fake, fake, 0, fq.LAYER_FUSED_CAST)
    assert lib.falqon_melded_forward_dump(C.byref(fused), fake, 0, None, 16, fake, 0, fake, fake, None, -1, fake, big, None) == inv
    assert lib.falqon_melded_forward_dump(C.byref(fused), fake, 0, None, 16, fake, 0, fake, fake, None, 2, fake, big, None) == inv   # 272 columns: blocks 0, 1
    assert lib.falqon_melded_forward_dump(C.byref(fused), fake, 1, None, 16, fake, 0, fake, fake, None, 0, fake, big, None) == fq.ERR_UNSUPPORTED   # fp32 X
    assert lib.falqon_melded_forward_dump(C.byref(layer), fake, 0, None, 16, fake, 0, fake, fake, None, 0, fake, big, None) == fq.ERR_UNSUPPORTED   # flag not set
    assert lib.falqon_melded_backward_dump(C.byref(fused), fake, 0, None, 16, fake, fake, fake, 0, fake, None, 1, fake, big, None) == inv   # 256 columns: block 0 only
    assert lib.falqon_melded_backward_dump(C.byref(fused), fake, 0, None, 16, fake, fake, None, 0, fake, None, 0, fake, big, None) == fq.ERR_UNSUPPORTED   # no dX
    assert fq.launch_count("falqon_melded_forward:fused") == 3 and fq.launch_count("falqon_melded_backward:fused") == 5
    bad_gran = fq.falqon_layer(256, 256, 16, fake, fake, fake, 2, 0)
    assert lib.falqon_melded_forward(C.byref(bad_gran), fake, 0, 16, fake, 0, fake, fake, None, fake, big, None) == inv
    odd = fq.falqon_layer(250, 256, 16, fake, fake, fake, 0, 0)
    assert lib.falqon_melded_forward(C.byref(odd), fake, 0, 16, fake, 0, fake, fake, None, fake, big, None) == inv
    # backward
    assert lib.falqon_melded_backward(C.byref(layer), fake, 0, 16, None, fake, fake, 0, fake, None, fake, big, None) == inv
    assert lib.falqon_melded_backward(C.byref(layer), fake, 0, 16, fake, fake, fake, 0, None, None, fake, big, None) == inv
    assert lib.falqon_melded_backward(C.byref(layer), fake, 0, 16, fake, fake, None, 0, fake, None, fake, 16, None) == wsp
    # proxy update
    assert lib.falqon_proxy_update(C.byref(layer), None, 0.1, 257, None, fake, big, None) == inv            # k > m
    assert lib.falqon_proxy_update(C.byref(layer), None, 0.1, -1, None, fake, big, None) == inv
    assert lib.falqon_proxy_update(C.byref(layer), None, float("nan"), 1, None, fake, big, None) == inv
    assert lib.falqon_proxy_update(C.byref(layer), None, 0.1, 1, None, fake, 64, None) == wsp
    assert lib.falqon_proxy_update(None, None, 0.1, 1, None, fake, big, None) == inv

    # batched proxy update: host arrays; any bad entry rejects the whole call
    two = (fq.falqon_layer * 2)(layer, fq.falqon_layer(128, 256, 8, fake + 0x100000, fake, fake + 0x200000, 0, 0))
    p2, i2, z2 = (C.c_void_p * 2), (C.c_int64 * 2), (C.c_size_t * 2)
    none2, ws2, big2 = p2(None, None), p2(fake + 0x300000, fake + 0x400000), z2(big, big)
    call = lib.falqon_proxy_update_batched
    assert call(two, 0, none2, 0.1, i2(1, 1), None, ws2, big2, None) == fq.OK                     # an empty call
    assert call(two, -1, none2, 0.1, i2(1, 1), None, ws2, big2, None) == inv
    assert call(None, 2, none2, 0.1, i2(1, 1), None, ws2, big2, None) == inv
    assert call(two, 2, none2, 0.1, i2(1, 129), None, ws2, big2, None) == inv                     # k > m in the second layer
    assert call(two, 2, none2, float("nan"), i2(1, 1), None, ws2, big2, None) == inv
    assert call(two, 2, none2, 0.1, i2(1, 1), None, p2(fake + 0x300000, fake + 0x300000), big2, None) == inv   # shared workspace
    assert call(two, 2, none2, 0.1, i2(1, 1), None, ws2, z2(big, 64), None) == wsp
    assert call(two, 2, none2, 0.1, i2(1, 1), None, p2(fake + 0x300000, None), big2, None) == wsp
    twice = (fq.falqon_layer * 2)(layer, layer)
    assert call(twice, 2, none2, 0.1, i2(1, 1), None, ws2, big2, None) == inv                     # the same layer twice
    # bounded-wait self-test: the limit must be 1..1000 ms
    assert lib.falqon_selftest_wait_timeout(0, None) == inv and lib.falqon_selftest_wait_timeout(1001, None) == inv
    # absmax
    assert lib.falqon_absmax(None, 0, 64, fake, fake, 8192, None) == inv
    assert lib.falqon_absmax(fake, 0, 0, fake, fake, 8192, None) == inv
    assert lib.falqon_absmax(fake, 5, 64, fake, fake, 8192, None) == inv
    assert lib.falqon_absmax(fake, 0, 64, None, fake, 8192, None) == inv
    assert lib.falqon_absmax(fake, 0, 64, fake, fake, 64, None) == wsp
    # tensor ceiling
    assert lib.falqon_tensor_ceiling(0, 1, 0, None, None, None, 0, 0, None) == inv
    assert lib.falqon_tensor_ceiling((1 << 20) + 1, 1, 0, None, None, None, 0, 0, None) == inv
    assert lib.falqon_tensor_ceiling(8, 1, 3, None, None, None, 0, 0, None) == inv                   # no such fill
    assert lib.falqon_tensor_ceiling(8, 1, 1, None, None, fake, 16384, 0, None) == inv               # stream buffer too small
    assert lib.falqon_tensor_ceiling(8, 1, 1, None, None, fake, 40000, 0, None) == inv            # not whole chunks
    assert lib.falqon_tensor_ceiling(8, 1, 1, None, None, fake, 65536, 8192, None) == inv         # fewer bytes per k-block than one tile


def test_launch_counts(fq):
    assert fq.launch_count("falqon_melded_forward") == 2
    assert fq.launch_count("falqon_melded_backward") == 2      # quantize (O_A cast riding), dX (dB riding)
    assert fq.launch_count("falqon_melded_backward:own_db") == 3
    assert fq.launch_count("falqon_proxy_update", k=4) == 2 and fq.launch_count("falqon_proxy_update", k=0) == 1
    assert fq.launch_count("falqon_proxy_update_batched", k=4) == 2 and fq.launch_count("falqon_proxy_update_batched", k=0) == 1
    assert fq.launch_count("nope") == 0


def test_headers_are_plain_c(tmp_path):
    """The ABI headers must compile as C99 (and as C++) on their own: no torch or CUDA types in the signatures."""
    import shutil
    import subprocess
    src = tmp_path / "use_headers.c"
    src.write_text('#include "falqon.h"\n#include "falqon_chain.h"\n'
                   "int main(void) { falqon_layer l; falqon_adamw h; (void)l; (void)h; return 0; }\n")
    inc = os.path.join(ROOT, "include")
    if shutil.which("gcc") is None:
        pytest.skip("no C compiler")
    subprocess.run(["gcc", "-std=c99", "-Wall", "-Wextra", "-pedantic", "-Werror", "-fsyntax-only", "-I", inc, str(src)], check=True)
    subprocess.run(["g++", "-std=c++11", "-Wall", "-Wextra", "-Werror", "-fsyntax-only", "-x", "c++", "-I", inc, str(src)], check=True)


def test_a_c_program_links_and_calls_the_library(tmp_path, fq):
    """A program written in C, built with gcc against the header and the shared library, calls the host-side entry
    points (no device needed): proof that the boundary is a C ABI and not a Python extension."""
    import shutil
    import subprocess
    if shutil.which("gcc") is None:
        pytest.skip("no C compiler")
    src = tmp_path / "client.c"
    src.write_text(r'''
#include <stdio.h>
#include "falqon.h"
int main(void) {
  size_t ws = falqon_workspace_bytes(4096, 4096, 64, 4096);
  size_t off = 0, size = 0;
  int rc = falqon_workspace_region(4096, 4096, 64, 4096, FALQON_WS_GQ, &off, &size);
  falqon_layer bad = {250, 256, 16, 0, 0, 0, FALQON_PER_TENSOR, 0};
  int inv = falqon_proxy_update(&bad, 0, 0.1f, 1, 0, 0, 0, 0);
  printf("%zu %d %zu %d %d\n", ws, rc, size, inv, falqon_launch_count("falqon_melded_backward", 0, 0, 0, 0, 0));
  return 0;
}
''')
    pkg = os.path.join(ROOT, "paper_2510_24061_b200")
    exe = tmp_path / "client"
    subprocess.run(["gcc", "-std=c99", "-Wall", "-Werror", "-I", os.path.join(ROOT, "include"), str(src), "-o", str(exe),
                    "-L", pkg, "-l:libfalqon.so", f"-Wl,-rpath,{pkg}"], check=True)
    out = subprocess.run([str(exe)], check=True, capture_output=True, text=True).stdout.split()
    assert int(out[0]) == fq.workspace_bytes(4096, 4096, 64, 4096) and int(out[0]) > 4096 * 4096
    assert int(out[1]) == fq.OK and int(out[2]) == 4096 * 4096
    assert int(out[3]) == fq.ERR_INVALID_ARG and int(out[4]) == 2


def test_the_package_refuses_to_load_without_its_library(tmp_path):
    """No CPU fallback: a copy of the Python package without libfalqon.so must fail at import, loudly."""
    import shutil
    import subprocess
    import sys
    pkg = tmp_path / "paper_2510_24061_b200"
    shutil.copytree(os.path.join(ROOT, "paper_2510_24061_b200"), pkg,
                    ignore=shutil.ignore_patterns("*.so", "build", "__pycache__", "csrc"))
    res = subprocess.run([sys.executable, "-c", "import paper_2510_24061_b200.binding"], cwd=tmp_path, capture_output=True,
                         text=True, env={**os.environ, "PYTHONPATH": str(tmp_path)})
    assert res.returncode != 0
    assert "ImportError" in res.stderr and "libfalqon.so is missing" in res.stderr and "no non-CUDA fallback" in res.stderr
    res = subprocess.run([sys.executable, "-c", "import paper_2510_24061_b200.stack"], cwd=tmp_path, capture_output=True,
                         text=True, env={**os.environ, "PYTHONPATH": str(tmp_path)})
    assert res.returncode != 0 and "ImportError" in res.stderr


def test_the_product_path_never_touches_the_oracle():
    """The oracle is test infrastructure: nothing in the package may import or execute it, and bench.py may do so only
    inside the function that times it (the cpu_baseline and reference legs)."""
    import ast
    pkg = os.path.join(ROOT, "paper_2510_24061_b200")
    for dirpath, _, files in os.walk(pkg):
        for name in files:
            if name.endswith((".py", ".cu", ".cuh", ".h", ".cpp")):
                text = open(os.path.join(dirpath, name)).read()
                if name.endswith(".py"):
                    for node in ast.walk(ast.parse(text)):
                        mods = []
                        if isinstance(node, ast.Import):
                            mods = [a.name for a in node.names]
                        elif isinstance(node, ast.ImportFrom):
                            mods = [node.module or ""]
                        assert not any(mod.split(".")[0] == "oracle" for mod in mods), f"{name} imports the oracle"
                else:
                    assert "oracle/" not in text and "falqon_oracle" not in text, f"{name} refers to the oracle"
    tree = ast.parse(open(os.path.join(ROOT, "bench.py")).read())
    importers = set()
    for fn in [n for n in ast.walk(tree) if isinstance(n, ast.FunctionDef)]:
        for node in ast.walk(fn):
            if isinstance(node, ast.ImportFrom) and (node.module or "").split(".")[0] == "oracle":
                importers.add(fn.name)
    top_level = [n for n in tree.body if isinstance(n, (ast.Import, ast.ImportFrom))]
    assert not any(getattr(n, "module", None) == "oracle" or any(a.name.startswith("oracle") for a in n.names) for n in top_level)
    assert importers == {"time_oracle_sample"}, importers
