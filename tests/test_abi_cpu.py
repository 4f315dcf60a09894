"""Host-side checks of the C ABI that need no GPU: the library loads, exports every declared symbol,
and its pure-host entry points behave."""
import ctypes
import re
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent


def _declared_symbols():
    text = (ROOT / "include" / "dodo.h").read_text()
    return re.findall(r"^DODO_API\s+[\w\s\*]+?\b(dodo_\w+)\s*\(", text, flags=re.M)


def test_header_declares_the_path():
    names = _declared_symbols()
    for required in ("dodo_score", "dodo_select", "dodo_score_select", "dodo_gather_kv", "dodo_attend"):
        assert required in names


def test_library_exports_every_declared_symbol(libdodo):
    lib = ctypes.CDLL(str(libdodo))
    for name in _declared_symbols():
        assert hasattr(lib, name), f"{name} is declared in dodo.h but not exported"


def test_binding_covers_every_declared_symbol(libdodo):
    from paper_2310_02409_b200 import api
    assert sorted(api.SIGNATURES) == sorted(_declared_symbols())
    api.load()


def test_num_nuggets_host_function(libdodo):
    from paper_2310_02409_b200 import api
    lib = api.load()
    golden = ROOT / "tests" / "golden" / "nugget_counts.txt"
    for line in golden.read_text().splitlines():
        line = line.split("#")[0].strip()
        if line:
            n, r, k = (int(x) for x in line.split())
            assert lib.dodo_num_nuggets(n, r) == k
    assert lib.dodo_num_nuggets(-1, 10) == -1 and lib.dodo_num_nuggets(10, 0) == -1
    assert lib.dodo_num_nuggets(0, 10) == 0


def test_num_nuggets_agrees_with_oracle(libdodo, oracle):
    from paper_2310_02409_b200 import api
    lib = api.load()
    for n in range(0, 400):
        for r in (1, 2, 3, 5, 10, 20, 33):
            assert lib.dodo_num_nuggets(n, r) == oracle.num_nuggets(n, r)


def test_create_without_gpu_fails_cleanly(libdodo):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    from paper_2310_02409_b200 import api
    with pytest.raises(api.DodoError) as e:
        api.Dodo(0)
    assert e.value.status == api.ERR_CUDA
