"""Host-side checks that need no GPU: the C-ABI library loads and exports every
symbol that include/zoa.h declares, and argument validation that happens before
any CUDA call works."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "zoa.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(zoa_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    from paper_2202_06009_b200 import binding
    names = _declared()
    assert len(names) >= 20
    lib = ctypes.CDLL(binding.LIB_PATH)
    for name in names:
        assert hasattr(lib, name), f"{name} is declared in include/zoa.h but not exported"
    assert set(names) == set(binding.EXPORTS), "binding and header disagree"


def test_header_is_plain_c(tmp_path):
    """The header compiles as C99 on its own: no C++ or torch types in the boundary."""
    import subprocess
    src = tmp_path / "t.c"
    src.write_text('#include "zoa.h"\nint main(void) { zoa_stats s; (void)s; return ZOA_OK; }\n')
    subprocess.check_call(["gcc", "-std=c99", "-Wall", "-Werror", "-I", os.path.join(ROOT, "include"),
                           "-c", str(src), "-o", str(tmp_path / "t.o")])


def test_validation_before_any_cuda_call():
    from paper_2202_06009_b200 import binding as B
    h = ctypes.c_void_p()
    for args in ((0, 2, 0.9, 0.999, 1e-8, 64), (10, 0, 0.9, 0.999, 1e-8, 64), (10, 65, 0.9, 0.999, 1e-8, 64),
                 (10, 2, 1.0, 0.999, 1e-8, 64), (10, 2, 0.9, -0.1, 1e-8, 64), (10, 2, 0.9, 0.999, 0.0, 64),
                 (10, 2, 0.9, 0.999, 1e-8, 33), (10, 2, 0.9, 0.999, 1e-8, 16), (10, 2, 0.9, 0.999, 1e-8, (1 << 30) + 32)):
        assert B.lib.zoa_create(ctypes.byref(h), *args) == B.ERR_ARG
        assert h.value is None and B.lib.zoa_last_error(None)
    assert B.lib.zoa_destroy(None) == B.ERR_ARG
    assert B.lib.zoa_sync_due(None, 0) < 0 and B.lib.zoa_var_due(None, 0) < 0
    assert B.lib.zoa_onebit_reduce(None, None) == B.ERR_ARG


def test_product_has_no_route_to_the_oracle():
    """Nothing under the package may import or name the oracle."""
    pkg = os.path.join(ROOT, "paper_2202_06009_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                assert "oracle" not in open(os.path.join(dirpath, f)).read().replace("test oracle", ""), f


def test_paper_schedules():
    """The T_v gap rule and the T_u interval rule of the paragraph "Policy for T_v and T_u",
    checked against values worked out by hand from the rules."""
    from paper_2202_06009_b200 import binding as B
    # kappa = 16: sixteen gaps of 1, sixteen of 2, sixteen of 4, ...
    steps = B.zoa_policy_var_steps(16, 200)
    assert steps[:17] == list(range(17))
    assert steps[17:33] == list(range(18, 49, 2)) and steps[33] == 52 and steps[34] == 56
    gaps = [b - a for a, b in zip(steps, steps[1:])]
    assert gaps[:16] == [1] * 16 and gaps[16:32] == [2] * 16 and set(gaps[32:48]) <= {4}
    assert steps[-1] < 200
    assert B.zoa_policy_var_steps(1, 40) == [0, 1, 3, 7, 15, 31]        # gaps 1, 2, 4, 8, 16
    assert B.zoa_policy_var_steps(16, 0) == []
    # BERT: interval 1 through the 12.5K warm-up, x2 every 32678 steps, clipped at 16
    b, k = B.zoa_policy_sync_pieces(12500, 32678, 16)
    assert k == [1, 2, 4, 8, 16]
    assert b == [0, 12500 + 32678, 12500 + 2 * 32678, 12500 + 3 * 32678, 12500 + 4 * 32678]
    assert B.zoa_policy_sync_pieces(10, 5, 1) == ([0], [1])
    assert B.zoa_policy_sync_pieces(0, 4, 12) == ([0, 4, 8, 12, 16], [1, 2, 4, 8, 12])
    assert B.lib.zoa_policy_sync_pieces(0, 0, 4, None, None, 0) == 0      # bad arguments
