"""The shared library loads without a GPU and exports every function the public
header declares; the ctypes mirrors have the sizes the header's structs have."""
import ctypes
import os
import re
import subprocess
import tempfile

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "condensa_cstep.h")


def declared_functions():
    text = open(HEADER).read()
    return re.findall(r"CONDENSA_API\s+[\w\s\*]+?\b(condensa_\w+)\s*\(", text)


def test_library_exports_every_declared_symbol():
    from paper_1911_02497_b200 import build, cstep
    build.build()
    names = declared_functions()
    assert len(names) >= 14 and "condensa_cstep_block" in names
    lib = ctypes.CDLL(cstep.LIB_PATH)
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(set(names)) == sorted(set(cstep.EXPORTS))


def test_struct_mirrors_match_the_header():
    """Compile a tiny C program against the header and compare sizeof."""
    from paper_1911_02497_b200 import cstep
    src = '#include <stdio.h>\n#include "condensa_cstep.h"\nint main(void){printf("%zu %zu %zu\\n",' \
          'sizeof(condensa_tensor),sizeof(condensa_result),sizeof(condensa_kernel_time));return 0;}\n'
    with tempfile.TemporaryDirectory() as d:
        c = os.path.join(d, "s.c")
        open(c, "w").write(src)
        exe = os.path.join(d, "s")
        subprocess.run(["gcc", "-I", os.path.join(ROOT, "include"), "-o", exe, c], check=True)
        sizes = [int(x) for x in subprocess.run([exe], capture_output=True, text=True, check=True).stdout.split()]
    assert sizes == [ctypes.sizeof(cstep.Tensor), ctypes.sizeof(cstep.Result), ctypes.sizeof(cstep.KernelTime)]


def test_calls_fail_loudly_without_a_device():
    import torch
    from paper_1911_02497_b200 import cstep
    if torch.cuda.is_available():
        return
    try:
        cstep.Context(0)
    except cstep.CondensaError as e:
        assert e.code == cstep.ERR_CUDA
    else:
        raise AssertionError("creating a context without a GPU must fail")
