"""The in-tree build when several ranks of one job import the package at once: one compiler
run, a complete library for everyone (a stand-in compiler and a scratch output path)."""
import os
import stat
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_concurrent_builds_compile_once(tmp_path):
    log = tmp_path / "runs.log"
    fake = tmp_path / "fake_nvcc"
    fake.write_text(textwrap.dedent(f"""\
        #!/bin/sh
        out=""
        while [ $# -gt 0 ]; do
          if [ "$1" = "-o" ]; then out="$2"; fi
          shift
        done
        echo run >> {log}
        sleep 1
        printf 'partial' > "$out"
        sleep 1
        printf 'complete library' > "$out"
        """))
    fake.chmod(fake.stat().st_mode | stat.S_IEXEC)
    child = textwrap.dedent(f"""\
        import os, sys
        sys.path.insert(0, {ROOT!r})
        from paper_1712_01887_b200 import build as b
        b.LIB = {str(tmp_path / "libfake.so")!r}
        os.environ["NVCC"] = {str(fake)!r}
        path = b.build()
        assert open(path).read() == "complete library", open(path).read()
        """)
    procs = [subprocess.Popen([sys.executable, "-c", child]) for _ in range(4)]
    assert [p.wait(timeout=60) for p in procs] == [0, 0, 0, 0]
    assert log.read_text().count("run") == 1
    assert not [f for f in os.listdir(tmp_path) if f.endswith(".tmp")]
