"""Host-only checks of the C ABI: the library loads without a GPU and exports what the header declares."""
import ctypes as C
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "uncomp.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(uncomp_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    from paper_2410_03090_b200 import build
    lib = C.CDLL(build.build())
    names = _declared()
    assert {"uncomp_entropy", "uncomp_assign_budgets", "uncomp_score_select", "uncomp_compact"} <= set(names)
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in uncomp.h but not exported"


def test_workspace_bytes_and_strerror_are_pure_host_functions():
    from paper_2410_03090_b200 import binding as ub
    ok = ub.make_shape(1, 32, 8, 32, 32768, 128, 64, "bf16")
    assert ub.uncomp_workspace_bytes(ok) > 0
    for bad in (ub.make_shape(1, 32, 8, 32, 32768, 64, 64, "bf16"),      # d != 128
                ub.make_shape(1, 32, 8, 30, 32768, 128, 64, "bf16"),     # Hq % H != 0
                ub.make_shape(1, 32, 8, 32, 64, 128, 64, "bf16"),        # N <= w
                ub.make_shape(1, 32, 8, 128, 4096, 128, 64, "bf16"),     # G * w > 512
                ub.make_shape(0, 32, 8, 32, 4096, 128, 64, "bf16")):
        assert ub.uncomp_workspace_bytes(bad) == 0
    assert ub.lib.uncomp_strerror(0) == b"ok"
    for code in range(-7, 0):
        assert len(ub.lib.uncomp_strerror(code)) > 0
    assert ub.lib.uncomp_version() >= 100


def test_product_package_does_not_touch_the_oracle():
    pkg = os.path.join(ROOT, "paper_2410_03090_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert "import oracle" not in src and "from oracle" not in src and "liboracle" not in src, f
