"""The C-ABI library builds, loads, and exports every function the public header declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    src = open(os.path.join(ROOT, "include", "mix.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(mix_[a-z_]+)\s*\(", src)))


def test_header_declares_the_boundary_calls():
    names = _declared()
    for must in ("mix_create", "mix_destroy", "mix_register_app", "mix_set_slot_map", "mix_apply",
                 "mix_register_sae_weights", "mix_get_status"):
        assert must in names


def test_library_builds_loads_and_exports_every_declared_symbol():
    from paper_2607_22595_b200 import _build
    path = _build.build()
    lib = ctypes.CDLL(path)
    for name in _declared():
        assert hasattr(lib, name), "libmix.so does not export %s" % name


def test_binding_lists_the_same_names_and_refuses_to_run_without_a_gpu():
    import torch
    import paper_2607_22595_b200 as mixlib
    assert sorted(mixlib.binding.EXPORTS) == _declared()
    if not torch.cuda.is_available():
        with pytest.raises(RuntimeError):
            mixlib.Mix(d_model=128, T_max=8, n_slots_max=2)          # no CPU fallback


def test_null_arguments_are_rejected_without_touching_a_device():
    import paper_2607_22595_b200 as mixlib
    lib = mixlib.load_library()
    assert lib.mix_create(None, None) == -1
    assert lib.mix_destroy(None) == 0
    assert lib.mix_apply(None, None, 0, None, None) == -1
    assert lib.mix_last_error(None) == b"null context"
