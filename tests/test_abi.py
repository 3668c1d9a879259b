"""The C-ABI library loads without a GPU and exports every symbol the header declares."""
import os
import re

from paper_2509_22323_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "rapid3.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(rapid3_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = binding.load()
    names = declared_symbols()
    assert len(names) >= 12
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(binding.EXPORTS) == names


def test_strerror_and_shape_helpers_run_on_the_host():
    assert binding.strerror(0) == "ok"
    assert "wait" in binding.strerror(-5)
    lib = binding.load()
    import ctypes
    s = binding.Shape(3, 24, 128, 512, 4096, 64, 24 * 4608 * 128, 4608 * 128, 128)
    assert lib.rapid3_num_blocks(ctypes.byref(s)) == 72
    assert lib.rapid3_mask_words(ctypes.byref(s)) == 2
    s2 = binding.Shape(2, 24, 64, 333, 4096, 64, 24 * 4429 * 64, 4429 * 64, 64)
    assert lib.rapid3_num_blocks(ctypes.byref(s2)) == 70
    bad = binding.Shape(1, 2, 96, 64, 256, 64, 1, 1, 96)
    assert lib.rapid3_num_blocks(ctypes.byref(bad)) == -2
    # (image, head) pairs index one grid dimension: more than 65535 of them is an unsupported shape
    wide = binding.Shape(64, 2048, 64, 64, 256, 64, 2048 * 320 * 64, 320 * 64, 64)
    assert lib.rapid3_num_blocks(ctypes.byref(wide)) == -2
    handle = ctypes.c_void_p()
    assert lib.rapid3_create(ctypes.byref(handle), ctypes.byref(wide)) == -2 and not handle.value


def test_null_context_is_refused_before_any_gpu_call():
    """Every entry point that takes a context returns RAPID3_ERR_INVALID_ARG (-1) for a NULL one: host-side
    argument checking runs before any CUDA call, so this holds without a GPU."""
    import ctypes
    lib = binding.load()
    one_i = (ctypes.c_int32 * 1)(2)
    one_f = (ctypes.c_float * 1)(0.5)
    null = None
    assert lib.rapid3_block_scores(null, null, null, null, 1, null, null) == -1
    assert lib.rapid3_select_mask(null, null, one_f, 1, null, null, null, null) == -1
    assert lib.rapid3_select_mask_mass(null, null, one_f, 1.0, 1, null, null, null, null, null) == -1
    assert lib.rapid3_sparse_joint_attn(null, null, null, null, null, null, 1, null, null, 1.0, null) == -1
    assert lib.rapid3_gated_step(null, null, null, null, null, one_i, one_f, 1, 1.0, null) == -1
    assert lib.rapid3_gated_step_heads(null, null, null, null, null, one_i, one_f, 1, 1.0, null) == -1
    assert lib.rapid3_gated_step_mass(null, null, null, null, null, one_i, one_f, 1.0, 1, 1.0, null) == -1
    assert lib.rapid3_gated_step_device(null, null, null, null, null, null, null, 1, 1.0, null) == -1
    assert lib.rapid3_gated_step_fused(null, null, null, null, null, null, null, 1e-6, null, null, null, one_i, one_f, 1,
                                       1.0, null) == -1
    assert lib.rapid3_gated_step_host(null, null, null, null, null, one_i, one_f, 1, 1.0, null, null, null) == -1
    assert lib.rapid3_debug_inject_timeout(null, null, null, null, null, 0, 1.0, null) == -1
    assert lib.rapid3_profile(null, 1) == -1
    assert lib.rapid3_launch_count(null) == -1
    assert lib.rapid3_destroy(null) in (0, -1)
