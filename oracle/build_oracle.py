"""Compiles the C oracle (test infrastructure) into oracle/_dsfacto_oracle.so with gcc."""
from __future__ import annotations

import os
import subprocess
from pathlib import Path

HERE = Path(__file__).resolve().parent
LIB_ORACLE = HERE / "_dsfacto_oracle.so"


def build_oracle(force: bool = False) -> Path:
    srcs = sorted(HERE.glob("*.c"))
    deps = srcs + sorted(HERE.glob("*.h"))
    stale = force or not LIB_ORACLE.exists() or any(p.stat().st_mtime > LIB_ORACLE.stat().st_mtime for p in deps)
    if stale:
        tmp = LIB_ORACLE.with_suffix(".so.tmp%d" % os.getpid())
        # -ffp-contract=off: every product and sum is rounded as written (no fused multiply-add)
        cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-ffp-contract=off", "-shared", "-fPIC", "-o", str(tmp)]
        cmd += [str(s) for s in srcs] + ["-lm"]
        proc = subprocess.run(cmd, capture_output=True, text=True)
        if proc.returncode != 0:
            raise RuntimeError("oracle build failed:\n" + proc.stdout + proc.stderr)
        os.replace(tmp, LIB_ORACLE)
    return LIB_ORACLE


if __name__ == "__main__":
    print(build_oracle(force=True))
