"""The C ABI used from plain C: include/sparbit.h must compile with a C compiler, and the host-only
entry points must behave as documented without a GPU."""
import subprocess
from pathlib import Path

ROOT = Path(__file__).resolve().parent.parent
LIBDIR = ROOT / "paper_2109_08751_b200"


def test_header_compiles_as_c_and_host_entry_points_work(tmp_path):
    exe = tmp_path / "abi_host_check"
    subprocess.run(["gcc", "-std=c99", "-Wall", "-Wextra", "-Werror", "-pedantic", f"-I{ROOT / 'include'}",
                    str(ROOT / "tests" / "c" / "abi_host_check.c"), "-o", str(exe), f"-L{LIBDIR}",
                    "-lsparbit_b200", f"-Wl,-rpath,{LIBDIR}"], check=True)
    r = subprocess.run([str(exe)], capture_output=True, text=True, timeout=60)
    assert r.returncode == 0, r.stderr
    assert "abi ok" in r.stdout
