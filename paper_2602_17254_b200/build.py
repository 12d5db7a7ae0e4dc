"""Builds ``libtrivance.so`` (the C-ABI library) in-tree with nvcc for sm_100a.

Usage: ``python -m paper_2602_17254_b200.build [--force] [--verbose]``

Every object is keyed by a hash of its compile command and of the code (comments and blank lines left out) of
its source and of every header that source includes, directly or not: an edit to a comment or to an unrelated
file recompiles nothing.
"""
import concurrent.futures
import hashlib
import os
import re
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libtrivance.so")
OBJ = os.path.join(HERE, "build")

# (source, extra flags, object name); the line-group kernel is compiled in parts (see its header comment)
UNITS = [(s, [], os.path.splitext(s)[0] + ".o") for s in (
    "trv_plan.cc", "trv_api.cu", "trv_host.cu", "trv_step.cu", "trv_step_gen.cu", "trv_fused_lat.cu", "trv_fused_t999.cu",
    "trv_fused_t999_tma.cu", "trv_fused_wide.cu", "trv_fused_bw.cu", "trv_fused_tree.cu", "trv_pipe.cu", "trv_pipe_bw.cu", "trv_linkloads.cu", "trv_noalloc.cu", "trv_joint.cu", "trv_comparator.cu")]
UNITS += [("trv_fused_lines.cu", ["-DTRV_LN_PART=%d" % k], "trv_fused_lines_p%d.o" % k) for k in range(5)]
SOURCES = sorted({u[0] for u in UNITS})
NVCC_FLAGS = ["-O3", "-std=c++17", "-lineinfo", "-gencode", "arch=compute_100a,code=sm_100a",
              "-Xcompiler", "-fPIC", "--expt-relaxed-constexpr"]

_INCLUDE = re.compile(r'^\s*#\s*include\s*"([^"]+)"', re.M)
_COMMENT = re.compile(r'//[^\n]*|/\*.*?\*/', re.S)


def _nvcc():
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.sep not in cand or os.path.exists(cand)):
            return cand
    raise RuntimeError("nvcc not found")


def _closure(path, seen):
    """path and every file it includes with quotes, transitively."""
    path = os.path.normpath(path)
    if path in seen or not os.path.exists(path):
        return
    seen.add(path)
    with open(path) as f:
        text = f.read()
    for inc in _INCLUDE.findall(text):
        _closure(os.path.join(os.path.dirname(path), inc), seen)


def _key(src, flags):
    files = set()
    _closure(os.path.join(CSRC, src), files)
    h = hashlib.sha256(" ".join(NVCC_FLAGS + flags).encode())
    for path in sorted(files):
        with open(path) as f:
            code = _COMMENT.sub("", f.read())
        h.update(os.path.basename(path).encode())
        h.update("\n".join(line.rstrip() for line in code.splitlines() if line.strip()).encode())
    return h.hexdigest()


def build(force=False, verbose=False):
    """Compile what changed for sm_100a and link the shared library.  Returns its path."""
    os.makedirs(OBJ, exist_ok=True)
    nvcc = _nvcc()
    extra = ["-Xptxas", "-v"] if verbose else []
    todo, objs = [], []
    for src, flags, name in UNITS:
        obj, key = os.path.join(OBJ, name), _key(src, flags)
        objs.append(obj)
        try:
            with open(obj + ".key") as f:
                fresh = os.path.exists(obj) and f.read().strip() == key
        except OSError:
            fresh = False
        if force or verbose or not fresh:
            todo.append((src, flags, obj, key))
    if not todo and os.path.exists(LIB) and all(os.path.getmtime(LIB) >= os.path.getmtime(o) for o in objs):
        return LIB

    def compile_one(job):
        src, flags, obj, key = job
        cmd = [nvcc] + NVCC_FLAGS + flags + extra + ["-x", "cu", "-c", os.path.join(CSRC, src), "-o", obj]
        r = subprocess.run(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)
        if r.returncode != 0:
            raise RuntimeError("nvcc failed on %s %s:\n%s" % (src, " ".join(flags), r.stdout))
        with open(obj + ".key", "w") as f:
            f.write(key)
        return r.stdout

    with concurrent.futures.ThreadPoolExecutor(max_workers=max(1, min(len(todo), os.cpu_count() or 4))) as ex:
        outputs = list(ex.map(compile_one, todo))
    if verbose:
        for out in outputs:
            sys.stdout.write(out)
    tmp = LIB + ".%d.tmp" % os.getpid()
    cmd = [nvcc, "-shared", "-o", tmp] + objs + ["-gencode", "arch=compute_100a,code=sm_100a"]
    r = subprocess.run(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)
    if r.returncode != 0:
        raise RuntimeError("link failed:\n%s" % r.stdout)
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
