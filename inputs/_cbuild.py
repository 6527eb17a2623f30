"""Compile one C file of this folder into a shared library beside it (gcc, on demand).

The library name carries a hash of the source and of the host CPU's feature
flags, so a library built on one machine is rebuilt rather than loaded on a
machine with a different CPU.
"""
import hashlib
import os
import subprocess


def _cpu_tag() -> str:
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.startswith("flags"):
                    return hashlib.sha1(line.encode()).hexdigest()[:8]
    except OSError:
        pass
    return "generic"


def build_shared(src_path: str, stem: str, extra_flags=()) -> str:
    src_path = os.path.abspath(src_path)
    with open(src_path, "rb") as f:
        digest = hashlib.sha1(f.read() + " ".join(extra_flags).encode()).hexdigest()[:10]
    out_dir = os.path.dirname(src_path)
    out = os.path.join(out_dir, f"lib{stem}_{digest}_{_cpu_tag()}.so")
    if os.path.exists(out):
        return out
    tmp = out + f".tmp{os.getpid()}"
    cmd = ["gcc", "-O2", "-std=c11", "-shared", "-fPIC", *extra_flags, src_path, "-o", tmp]
    subprocess.run(cmd, check=True)
    os.replace(tmp, out)
    return out
