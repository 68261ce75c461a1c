"""The shared library loads and exports every symbol the public header declares (no GPU needed)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADERS = [os.path.join(ROOT, "include", f) for f in sorted(os.listdir(os.path.join(ROOT, "include"))) if f.endswith(".h")]


def declared_symbols():
    text = "".join(open(h).read() for h in HEADERS)
    return sorted(set(re.findall(r"ET_API[^;(]*?\b(et_[a-z0-9_]+)\s*\(", text)))


@pytest.fixture(scope="module")
def built_lib():
    from paper_2605_30010_b200 import build
    return build.build()


def test_header_declares_the_boundary_calls():
    syms = declared_symbols()
    for need in ("et_encoder_create", "et_encode_video", "et_encode_batch", "et_destroy"):
        assert need in syms
    assert len(syms) >= 15


def test_library_exports_every_declared_symbol(built_lib):
    lib = ctypes.CDLL(built_lib)
    for s in declared_symbols():
        assert hasattr(lib, s), f"{s} is declared in include/*.h but not exported"


def test_binding_covers_every_declared_symbol(built_lib):
    from paper_2605_30010_b200 import binding
    assert sorted(binding.EXPORTS) == declared_symbols()
    for s in declared_symbols():
        assert hasattr(binding, s) or s in ("et_status_string", "et_last_error", "et_llm_last_error"), s


def test_struct_sizes_match_the_header(built_lib, tmp_path):
    """Compile a tiny C program against the header and compare sizeof() with the ctypes mirrors."""
    import subprocess
    from paper_2605_30010_b200 import binding as b
    src = tmp_path / "sz.c"
    src.write_text('#include <stdio.h>\n#include "earlytom_llm.h"\nint main(){printf("%zu %zu %zu %zu %zu %zu %zu %zu %zu %zu %zu\\n",'
                   'sizeof(et_config),sizeof(et_weights),sizeof(et_forced_plan),sizeof(et_params),sizeof(et_trace),'
                   'sizeof(et_result),sizeof(et_host_buffers),sizeof(et_llm_config),sizeof(et_llm_weights),'
                   'sizeof(et_llm_result),sizeof(et_llm_profile));return 0;}\n')
    exe = tmp_path / "sz"
    subprocess.check_call(["gcc", "-I", os.path.join(ROOT, "include"), str(src), "-o", str(exe)])
    sizes = [int(x) for x in subprocess.check_output([str(exe)]).split()]
    mine = [ctypes.sizeof(t) for t in (b.et_config, b.et_weights, b.et_forced_plan, b.et_params, b.et_trace,
                                       b.et_result, b.et_host_buffers, b.et_llm_config, b.et_llm_weights,
                                       b.et_llm_result, b.et_llm_profile)]
    assert sizes == mine


def test_no_gpu_calls_fail_cleanly(built_lib):
    """Without a device the create call reports ET_ERR_CUDA instead of computing anything on the CPU."""
    import numpy as np
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    from paper_2605_30010_b200 import binding as b
    from synthetic import EncoderShape, make_weights
    shape = EncoderShape(image_size=28, patch_size=14, num_layers=1, hidden=16, heads=2, mlp_dim=32)
    with pytest.raises(b.EarlyTomError) as ei:
        b.Encoder(shape, make_weights(shape, 0), b.ET_F32, 2)
    assert ei.value.status == 5
    # argument validation happens before any device work
    bad = b.et_config(28, 14, 1, 15, 2, 32, 1e-6, 1, 1, 0, 2, 1)
    w = np.zeros(4, dtype=np.float32)
    with pytest.raises(b.EarlyTomError) as ei:
        b.et_encoder_create(bad, w)
    assert ei.value.status == 2
