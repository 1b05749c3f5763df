"""AddressSanitizer + UndefinedBehaviorSanitizer over the host code: the oracle (``oracle/sw_oracle.c``) and the library's
host-only sources (controller, telemetry, error text) are rebuilt with ``-fsanitize=address,undefined`` and the CPU test
files that exercise them are replayed in a child process that has the sanitizer runtimes preloaded.  Any report is
fatal there, so a clean exit means a clean run."""
import subprocess
import sys
from pathlib import Path

ROOT = Path(__file__).resolve().parent.parent
REPLAYED = ["tests/test_controller.py", "tests/test_telemetry.py", "tests/test_oracle_chooser.py",
            "tests/test_oracle_first_fit.py", "tests/test_oracle_telemetry.py", "tests/test_oracle_attention.py",
            "tests/test_abi.py"]


def test_host_code_is_clean_under_asan_and_ubsan():
    from oracle import sw_oracle
    from paper_2609_07883_b200 import build

    lib = build.build_sanitized()
    sw_oracle.build(sanitize=True)
    env = build.sanitizer_env()
    env["SLOWEAVE_LIB"] = str(lib)
    env["SW_ORACLE_SANITIZE"] = "1"
    proc = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-p", "no:cacheprovider", *REPLAYED], cwd=ROOT, env=env,
                          stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True, timeout=1500)
    tail = proc.stdout[-4000:]
    assert proc.returncode == 0, tail
    assert "AddressSanitizer" not in proc.stdout and "runtime error" not in proc.stdout, tail
    assert " passed" in proc.stdout, tail
