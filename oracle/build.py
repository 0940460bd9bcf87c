"""Compile the C oracle with gcc into oracle/_build/.  Test infrastructure only."""
from __future__ import annotations

import os
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(_HERE, "alcs_oracle.c")
BUILD_DIR = os.path.join(_HERE, "_build")


def lib_path(mutant: int = 0, build_dir: str | None = None) -> str:
    name = "liboracle.so" if mutant == 0 else f"liboracle_mutant{mutant}.so"
    return os.path.join(build_dir or BUILD_DIR, name)


def build(mutant: int = 0, build_dir: str | None = None, force: bool = False) -> str:
    """Build (if stale) and return the path of the oracle shared object.

    The oracle is compiled as it stands: -O2, OpenMP over (image, output channel), no
    hand tuning.  `mutant` != 0 compiles one of the deliberately wrong variants that the
    pin tests use to show they can tell a wrong oracle from the right one.
    """
    out = lib_path(mutant, build_dir)
    os.makedirs(os.path.dirname(out), exist_ok=True)
    if not force and os.path.exists(out) and os.path.getmtime(out) >= os.path.getmtime(SRC):
        return out
    tmp = out + f".tmp{os.getpid()}"
    cmd = ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-Wall", "-Wextra",
           f"-DORACLE_MUTANT={mutant}", SRC, "-o", tmp, "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, out)
    return out


if __name__ == "__main__":
    print(build(force=True))
