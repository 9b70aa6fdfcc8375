"""The C-ABI library builds for sm_100a without a GPU, loads, and exports what the header declares."""
import os
import re

import paper_2502_01662_b200 as pkg

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "cos_verify.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(cos_verify_\w+)\s*\(", text)))


def test_every_declared_symbol_is_exported():
    lib = pkg.load_library()
    names = _declared()
    assert "cos_verify_create" in names and "cos_verify_run" in names and "cos_verify_destroy" in names
    for name in names:
        assert hasattr(lib, name), name


def test_create_validates_before_touching_the_device():
    # host-side validation runs first, so these fail the same way with or without a GPU
    for kw in (dict(n=0), dict(n=9), dict(weights=[0.7, 0.7]), dict(temperature=-1.0), dict(vocab=0),
               dict(gamma=-1), dict(combine=0, mask_model=0), dict(cluster_size=3)):
        args = dict(n=2, combine=0, weights=[0.5, 0.5], temperature=1.0, gamma=2, vocab=100, max_batch=2,
                    dtype=pkg.COS_DTYPE_F32)
        args.update(kw)
        try:
            pkg.CosVerifier(**args)
        except pkg.CosVerifyError as e:
            assert e.status == 1, (kw, e)
        else:
            raise AssertionError(f"accepted {kw}")


def test_binding_constants_are_the_headers():
    """Every COS_* enumerator of the header has the same value in the binding (flags, status codes, row bits)."""
    from paper_2502_01662_b200 import binding
    with open(os.path.join(ROOT, "include", "cos_verify.h")) as f:
        text = re.sub(r"/\*.*?\*/", "", f.read(), flags=re.S)
    found = {}
    for name, value in re.findall(r"\b(COS_[A-Z0-9_]+)\s*=\s*([^,}\n]+)", text):
        value = value.strip()
        m = re.fullmatch(r"(\d+)u?\s*<<\s*(\d+)", value)
        found[name] = (int(m.group(1)) << int(m.group(2))) if m else int(value.rstrip("u"), 0)
    assert len(found) >= 20, found
    checked = 0
    for name, value in found.items():
        if hasattr(binding, name):
            assert getattr(binding, name) == value, (name, getattr(binding, name), value)
            checked += 1
    for name in ("COS_RUN_ALL_RESIDUALS", "COS_RUN_PROPOSER_PER_POSITION", "COS_RUN_BONUS_FROM_MODEL", "COS_RUN_EARLY_EXIT",
                 "COS_RUN_INPUTS_SETTLED", "COS_ROW_FAULT", "COS_ROW_NONFINITE"):
        assert name in found and hasattr(binding, name), name
    assert checked >= 12, checked
