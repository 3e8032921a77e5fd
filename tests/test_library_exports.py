"""The C-ABI library loads without a GPU and exports every symbol the header declares."""
import os
import re

from paper_2012_04201_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "bbo_mlp_cv.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(bbo_mlp_cv_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported():
    lib = binding.load()
    names = declared_symbols()
    assert len(names) >= 14
    for name in names:
        assert hasattr(lib, name), name
    assert sorted(binding.EXPORTS) == names


def test_strerror_and_argument_checks_without_a_device():
    lib = binding.load()
    assert lib.bbo_mlp_cv_strerror(0) == b"ok"
    assert b"invalid" in lib.bbo_mlp_cv_strerror(binding.BBO_ERR_INVALID_ARG)
    assert lib.bbo_mlp_cv_create(None, None) == binding.BBO_ERR_INVALID_ARG
    assert lib.bbo_mlp_cv_destroy(None) == binding.BBO_ERR_INVALID_ARG
    assert lib.bbo_mlp_cv_eval(None, None, None, 0, 0, 0, 0, None, 0, 0, None) == binding.BBO_ERR_INVALID_ARG
    assert lib.bbo_mlp_cv_eval_holdout(None, None, None, 0, None, None, 0, 0, 0, None, 0, 0, None) == binding.BBO_ERR_INVALID_ARG


def test_config_layout_matches_header():
    from paper_2012_04201_b200.workloads import CONFIG_DTYPE
    assert CONFIG_DTYPE.itemsize == 32
    assert list(CONFIG_DTYPE.names) == ["hidden", "batch_size", "epochs", "alpha", "lr", "beta1", "beta2", "eps"]
    assert [CONFIG_DTYPE.fields[n][1] for n in CONFIG_DTYPE.names] == [0, 4, 8, 12, 16, 20, 24, 28]
