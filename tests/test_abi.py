"""The C-ABI library builds, loads without a GPU, and exports every symbol the header declares."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "tweo.h")).read()
    return re.findall(r"TWEO_API\s+[\w\s\*]+?\b(tweo_\w+)\s*\(", text)


def test_library_exports_every_declared_symbol():
    from paper_2511_23225_b200 import binding, build
    path = build.build()
    lib = ctypes.CDLL(path)
    names = declared_functions()
    assert len(names) >= 13 and len(set(names)) == len(names)
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in tweo.h but not exported"
    assert sorted(set(binding.EXPORTS)) == sorted(set(names))


def test_host_side_helpers_without_a_gpu():
    from paper_2511_23225_b200 import binding
    L = binding.lib()
    assert L.tweo_version() >= 100
    assert L.tweo_status_string(0) == b"ok"
    assert b"align" in L.tweo_status_string(3)
    assert L.tweo_workspace_bytes(binding.OP_QUANTIZE, 1 << 20, 0, 0) == 65536
    assert L.tweo_workspace_bytes(binding.OP_LOSS, 1 << 20, 12, 0) >= 256 + 8 * 12
    # argument validation happens on the host, before any CUDA call
    assert L.tweo_loss_fwd_bwd(None, 1, 8, 3.0, 1e-6, 4.0, 1.0, None, None, None, 0, None, 0, None) == 1
    assert L.tweo_quantize_per_tensor(None, -1, 0, 0, None, None, None, None, None, None, 0, None) == 1
    assert L.tweo_quantize_per_tensor_batch(None, 1, None, 0, None) == 1
    assert L.tweo_fp8_linear_fwd(None, 0, None, 0, None, None, None, 0, 1, 1, 1, 0, 0, None, None, 0, None) == 1


def test_binding_refuses_cpu_tensors():
    import pytest
    import torch
    from paper_2511_23225_b200 import binding
    with pytest.raises(TypeError):
        binding.quantize_per_tensor(torch.zeros(16, dtype=torch.bfloat16))


def test_tweo_log_dumps_the_arguments_of_a_call():
    """TWEO_LOG=1: every entry point prints its name and scalar arguments to stderr before anything else -- also for a
    call that the argument check then rejects, which is what can run without a GPU."""
    import subprocess
    import sys
    code = (
        "from paper_2511_23225_b200 import binding\n"
        "L = binding.lib()\n"
        "print(L.tweo_fp8_linear_fwd(None, 768, None, 768, None, None, None, 2304, 8192, 2304, 768, 0, 1, None, None, 0, None))\n"
        "print(L.tweo_fp4_unpack(None, 4096, None, None))\n")
    for env_value, expect in (("1", True), ("0", False), (None, False)):
        env = dict(os.environ)
        env.pop("TWEO_LOG", None)
        if env_value is not None:
            env["TWEO_LOG"] = env_value
        r = subprocess.run([sys.executable, "-c", code], cwd=ROOT, env=env, capture_output=True, text=True, timeout=300)
        assert r.returncode == 0 and r.stdout.split() == ["1", "1"]            # both rejected: NULL operands
        logged = "[tweo] tweo_fp8_linear_fwd M=8192 N=2304 K=768 fmt_x=0 fmt_w=1 ldx=768 ldw=768 ldy=2304" in r.stderr
        assert logged == expect
        assert ("[tweo] tweo_fp4_unpack" in r.stderr and "n=4096" in r.stderr) == expect
