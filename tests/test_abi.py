"""The C-ABI library loads and exports every symbol include/*.h declares (no GPU needed)."""
import ctypes
import glob
import os
import re

import pytest

import paper_2101_05453_b200 as qlstm
from paper_2101_05453_b200 import binding
from workloads import make_workload

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    names = set()
    for path in glob.glob(os.path.join(ROOT, "include", "*.h")):
        text = re.sub(r"/\*.*?\*/", "", open(path).read(), flags=re.S)
        names |= set(re.findall(r"\b(qlstm_[a-z_0-9]+)\s*\(", text))
    return sorted(names)


def test_header_symbols_are_exported():
    names = declared_symbols()
    assert len(names) >= 10
    lib = ctypes.CDLL(qlstm.library_path()) if os.path.exists(qlstm.library_path()) else qlstm.lib()
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(binding.EXPORTS) == names


def test_strerror_covers_all_codes():
    for code in range(0, -8, -1):
        assert qlstm.strerror(code) and qlstm.strerror(code) != "unknown error"
    assert qlstm.strerror(-99) == "unknown error"


def test_create_fails_loudly_without_a_device():
    try:
        import torch
        if torch.cuda.is_available():
            pytest.skip("a CUDA device is present")
    except ImportError:
        pass
    w = make_workload(1)
    with pytest.raises(qlstm.QlstmError) as e:
        qlstm.QLSTM(w.layers, 4, 1)
    assert e.value.code == qlstm.ERR_CUDA


def test_argument_validation_precedes_device_use():
    w = make_workload(1)
    with pytest.raises(qlstm.QlstmError) as e:
        qlstm.QLSTM(w.layers, 0, 1)
    assert e.value.code == qlstm.ERR_ARG
    import copy
    bad = copy.copy(w.layers[0])
    bad.n_output = 7
    with pytest.raises(qlstm.QlstmError) as e:
        qlstm.QLSTM([bad], 4, 1)
    assert e.value.code == qlstm.ERR_DIM
