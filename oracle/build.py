"""Compile the scalar C oracle into oracle/libmqg_oracle.so with gcc.

Test infrastructure: building the checker is not using it.  No -march flags, so
the shared object runs on any x86-64 host it is copied to; fmaf comes from libm.
"""
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "mqg_oracle.c")
LIB = os.path.join(HERE, "libmqg_oracle.so")

FLAGS = ["-O2", "-std=c99", "-ffp-contract=off", "-fno-fast-math", "-fPIC", "-shared",
         "-Wall", "-Wextra"]


def build(force: bool = False) -> str:
    override = os.environ.get("MQG_ORACLE_LIB")      # the mutation tests load a planted copy
    if override:
        return override
    if (not force and os.path.exists(LIB)
            and os.path.getmtime(LIB) >= os.path.getmtime(SRC)):
        return LIB
    tmp = LIB + ".tmp.%d" % os.getpid()
    subprocess.run(["gcc", *FLAGS, "-o", tmp, SRC, "-lm"], check=True)
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force=True))
