"""Builds and runs csrc/tma_probe.cu: the TMA operand-streaming probe behind the GEMM kernel's stage layout.

    python -m paper_2609_31551_b200.tma_probe

Needs nvcc and a B200; prints one line per variant (time, bytes per second into the SMs, time per k-step and CTA)."""
from __future__ import annotations
import os
import subprocess
import sys
import tempfile

HERE = os.path.dirname(os.path.abspath(__file__))


def build(out_path: str) -> None:
    src = os.path.join(HERE, "csrc", "tma_probe.cu")
    cmd = ["nvcc", "-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-o", out_path, src, "-lcuda"]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)


def main() -> int:
    with tempfile.TemporaryDirectory() as tmp:
        exe = os.path.join(tmp, "tma_probe")
        build(exe)
        return subprocess.run([exe]).returncode


if __name__ == "__main__":
    sys.exit(main())
