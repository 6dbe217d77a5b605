"""Compile the C oracle into a shared object next to its source.

Test infrastructure only: nothing in the product package may import this.
"""
from __future__ import annotations

import os
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
SOURCE = os.path.join(_HERE, "adammini_oracle.c")
LIBRARY = os.path.join(_HERE, "liboracle_adammini.so")

# No fast-math and no FMA contraction: the sums must run left to right in
# plain IEEE float64, exactly as the source reads.
CFLAGS = ["-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math", "-fPIC", "-shared"]


def build(force: bool = False, source: str = SOURCE, library: str = LIBRARY) -> str:
    """Build `library` from `source` with gcc if it is missing or stale."""
    stale = (
        force
        or not os.path.exists(library)
        or os.path.getmtime(library) < os.path.getmtime(source)
    )
    if stale:
        tmp = library + f".tmp{os.getpid()}"
        subprocess.run(["gcc", *CFLAGS, "-o", tmp, source, "-lm"], check=True)
        os.replace(tmp, library)
    return library


if __name__ == "__main__":
    print(build(force=True))
