"""The oracle's own unit tests once more against a build of ``oracle/mip_oracle.c`` with gcc's address
and undefined-behaviour sanitizers: an index past a buffer or a signed overflow inside the oracle aborts
the child process instead of going unnoticed.  CPU only."""
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_oracle_pins_pass_under_asan_and_ubsan():
    from oracle import mip_oracle as orc
    env = orc.sanitizer_env()
    if not os.path.exists(env["LD_PRELOAD"]):
        import pytest
        pytest.skip("gcc has no libasan here")
    out = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-p", "no:cacheprovider",
                          os.path.join(ROOT, "tests", "test_oracle_pins.py"),
                          os.path.join(ROOT, "tests", "test_paper_isa_semantics.py")],
                         cwd=ROOT, env=env, capture_output=True, text=True, timeout=1500)
    assert out.returncode == 0, (out.stdout[-3000:], out.stderr[-3000:])
    assert " passed" in out.stdout and "failed" not in out.stdout
    assert os.path.exists(os.path.join(ROOT, "oracle", "libmip_oracle_san.so"))
