"""include/psa.h compiled as plain C (gcc -std=c11 -Wall -Wextra -Werror -pedantic) and the host-side entry
points called from a C program linked against libpsa.so: no Python between the caller and the ABI."""
import os
import subprocess

from paper_2410_20305_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_c_program_calls_the_host_side_entry_points(tmp_path):
    B.load_library()   # builds libpsa.so if the sources are newer
    libdir = os.path.join(ROOT, "paper_2410_20305_b200")
    exe = str(tmp_path / "c_abi_host")
    build = subprocess.run(["gcc", "-std=c11", "-Wall", "-Wextra", "-Werror", "-pedantic", "-I", os.path.join(ROOT, "include"),
                            os.path.join(ROOT, "tests", "c_abi_host.c"), "-o", exe, "-L", libdir, "-lpsa",
                            "-Wl,-rpath," + libdir], capture_output=True, text=True)
    assert build.returncode == 0, build.stderr
    run = subprocess.run([exe], capture_output=True, text=True, timeout=120)
    assert run.returncode == 0 and "C_ABI_OK" in run.stdout, run.stdout + run.stderr
