"""Builds libdragon.so in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
import os
import subprocess
import sys

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libdragon.so")
SOURCES = ["prune.cpp", "lower.cpp", "codegen.cpp", "specialize.cpp", "verify.cpp", "api.cu", "workspace.cu", "vm_launch.cu", "row_kernels.cu", "gemm_tcgen05.cu"]
NVCC = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "-Xcompiler", "-fPIC",
         "--expt-relaxed-constexpr", "-Xcompiler", "-Wall"] + os.environ.get("DRAGON_NVCC_DEFS", "").split()


def _stale(target, deps):
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(d) > t for d in deps)


def build(verbose=False, force=False, ptxas_info=False):
    objdir = os.path.join(HERE, "_build")
    os.makedirs(objdir, exist_ok=True)
    headers = [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith(".h")]
    headers.append(os.path.join(os.path.dirname(HERE), "include", "dragon.h"))
    objs = []
    for src in SOURCES:
        path = os.path.join(CSRC, src)
        obj = os.path.join(objdir, src + ".o")
        objs.append(obj)
        if force or ptxas_info or _stale(obj, [path] + headers):
            cmd = [NVCC] + FLAGS + (["-Xptxas", "-v"] if ptxas_info else []) + ["-x", "cu", "-c", path, "-o", obj]
            if verbose:
                print(" ".join(cmd), flush=True)
            subprocess.run(cmd, check=True)
    objs.append(_generated_kernel_object(objdir, verbose, force or ptxas_info))
    objs.append(_generated_templates_object(objdir, verbose, force))
    if force or _stale(LIB, objs):
        cmd = [NVCC, "-shared", "-o", LIB] + objs + ["-gencode", "arch=compute_100a,code=sm_100a"]
        if verbose:
            print(" ".join(cmd), flush=True)
        subprocess.run(cmd, check=True)
    return LIB


def _embed(cpp, obj, symbol, data, what):
    with open(cpp, "w") as fh:
        fh.write("// generated: %s\n" % what)
        fh.write('extern "C" const unsigned long %s_size = %d;\n' % (symbol, len(data)))
        fh.write('extern "C" const unsigned char %s[] = {' % symbol)
        fh.write(",".join(str(b) for b in data) if data else "0")
        fh.write("};\n")
    subprocess.run(["g++", "-O1", "-fPIC", "-c", cpp, "-o", obj], check=True)


def _generated_kernel_object(objdir, verbose, force):
    """vm_ptxgen.py -> PTX -> cubin of the graph-VM kernel, embedded as a byte array."""
    from paper_1707_08265_b200 import vm_ptxgen
    ptx, cubin = os.path.join(objdir, "vm_gen.ptx"), os.path.join(objdir, "vm_gen.cubin")
    cpp, obj = os.path.join(objdir, "vm_gen_cubin.cpp"), os.path.join(objdir, "vm_gen_cubin.o")
    if not (force or _stale(obj, [vm_ptxgen.__file__])):
        return obj
    open(ptx, "w").write(vm_ptxgen.generate())
    ptxas = os.path.join(os.path.dirname(NVCC), "ptxas")
    r = subprocess.run([ptxas, "-arch=sm_100a", "-O3", "-v", ptx, "-o", cubin], check=True, capture_output=True, text=True)
    if verbose:
        print(r.stderr, flush=True)
    _embed(cpp, obj, "dragon_vm_gen_cubin", open(cubin, "rb").read(), "cubin of the PTX-generated VM kernel")
    return obj


def _generated_templates_object(objdir, verbose, force):
    """vm_ptxgen.py -> the leaves of the VM kernel as PTX text (C++ string tables) for csrc/specialize.cpp."""
    from paper_1707_08265_b200 import vm_ptxgen
    cpp, obj = os.path.join(objdir, "vm_templates.cpp"), os.path.join(objdir, "vm_templates.o")
    if not (force or _stale(obj, [vm_ptxgen.__file__, os.path.join(CSRC, "vm_templates.h")])):
        return obj
    open(cpp, "w").write(vm_ptxgen.templates_source())
    cmd = ["g++", "-std=c++17", "-O0", "-fPIC", "-I", CSRC, "-c", cpp, "-o", obj]
    if verbose:
        print(" ".join(cmd), flush=True)
    subprocess.run(cmd, check=True)
    return obj


HOST_SOURCES = ["prune.cpp", "lower.cpp", "codegen.cpp", "specialize.cpp", "verify.cpp"]     # the host compiler: no CUDA in these
SAN_LIB = os.path.join(HERE, "libdragon_san.so")


def build_sanitized(verbose=False):
    """libdragon_san.so: the same library with the host compiler (prunes, lowering, code generation) built
    with -fsanitize=address,undefined.  Load it with DRAGON_LIB=<path> and the sanitizer runtime preloaded
    (LD_PRELOAD=$(gcc -print-file-name=libasan.so)); used by tests/test_sanitized_host_compiler.py."""
    build(verbose=verbose)
    objdir = os.path.join(HERE, "_build")
    headers = [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith(".h")]
    objs = []
    for src in SOURCES:
        if src not in HOST_SOURCES:
            objs.append(os.path.join(objdir, src + ".o"))
            continue
        path, obj = os.path.join(CSRC, src), os.path.join(objdir, src + ".san.o")
        objs.append(obj)
        if _stale(obj, [path] + headers):
            cmd = ["g++", "-std=c++17", "-O1", "-g", "-fPIC", "-fno-omit-frame-pointer", "-fsanitize=address,undefined",
                   "-fno-sanitize-recover=undefined", "-Wall", "-c", path, "-o", obj]
            if verbose:
                print(" ".join(cmd), flush=True)
            subprocess.run(cmd, check=True)
    objs.append(os.path.join(objdir, "vm_gen_cubin.o"))
    objs.append(os.path.join(objdir, "vm_templates.o"))
    if _stale(SAN_LIB, objs):
        cmd = [NVCC, "-shared", "-o", SAN_LIB] + objs + ["-gencode", "arch=compute_100a,code=sm_100a", "-Xcompiler", "-fsanitize=address", "-Xcompiler", "-fsanitize=undefined"]
        if verbose:
            print(" ".join(cmd), flush=True)
        subprocess.run(cmd, check=True)
    return SAN_LIB


if __name__ == "__main__":
    if "--sanitize" in sys.argv:
        print(build_sanitized(verbose=True))
    else:
        build(verbose=True, force="--force" in sys.argv, ptxas_info="--ptxas" in sys.argv)
