"""The C-ABI library loads without a GPU and exports every symbol the header declares (no compute calls)."""
import ctypes as C
import os
import re

from paper_2607_22648_b200 import build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "ptstore.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ptstore_[a-z_]+)\s*\(", text)))


def test_header_symbols_are_exported():
    lib = C.CDLL(build.build())
    names = declared_functions()
    assert len(names) >= 13
    for n in names:
        assert hasattr(lib, n), n


def test_binding_declares_the_same_entry_points():
    src = open(os.path.join(ROOT, "paper_2607_22648_b200", "binding.py")).read()
    listed = set(re.findall(r'"(ptstore_[a-z_]+)"', src))
    assert set(declared_functions()) <= listed


def test_host_only_calls_validate_arguments():
    from paper_2607_22648_b200.binding import Config
    lib = C.CDLL(build.build())
    lib.ptstore_workspace_bytes.restype = C.c_uint64
    lib.ptstore_workspace_bytes.argtypes = [C.POINTER(Config)]
    lib.ptstore_strerror.restype = C.c_char_p
    cfg = Config()
    assert lib.ptstore_workspace_bytes(C.byref(cfg)) == 0                      # struct_size not set
    cfg = Config(C.sizeof(Config), 0, 32, 8, 128, 2, 16, 64, 64 * 391, 0, None, None, 20000, 0, 28572, None, 0, 0, 0)
    need = lib.ptstore_workspace_bytes(C.byref(cfg))
    assert 1 << 20 < need < 1 << 26                                            # a few MB of metadata for 20k blocks
    cfg.table_slots = 20000                                                    # table must be larger than the pool
    assert lib.ptstore_workspace_bytes(C.byref(cfg)) == 0
    cfg.table_slots = 28572
    cfg.block_tokens, cfg.num_kv_heads, cfg.head_dim = 1, 1, 3                 # chunk of 6 bytes: not a multiple of 16
    assert lib.ptstore_workspace_bytes(C.byref(cfg)) == 0
    out = C.c_void_p()
    lib.ptstore_create.argtypes = [C.POINTER(Config), C.POINTER(C.c_void_p), C.c_void_p]
    assert lib.ptstore_create(C.byref(cfg), C.byref(out), None) == -1 and not out.value
    assert lib.ptstore_strerror(-1) == b"invalid argument"
    assert lib.ptstore_strerror(0) == b"ok"


def test_header_is_plain_c():
    """The boundary is a C ABI: the header must compile as C99 with no other include than stdint.h."""
    import subprocess
    import tempfile
    src = '#include "ptstore.h"\nint main(void) { ptstore_config_t c; c.struct_size = (uint32_t)sizeof c; return (int)(c.struct_size == 0) + PTSTORE_OK; }\n'
    with tempfile.TemporaryDirectory() as d:
        path = os.path.join(d, "t.c")
        open(path, "w").write(src)
        subprocess.check_call(["gcc", "-std=c99", "-Wall", "-Wextra", "-Werror", "-pedantic", "-I", os.path.join(ROOT, "include"),
                               "-fsyntax-only", path])


def test_ctypes_structs_match_the_c_layout():
    """sizeof / offsetof of the structs the binding declares, checked against the C compiler."""
    import subprocess
    import tempfile
    from paper_2607_22648_b200.binding import Config, PagedCache, Stats
    prog = r'''
#include <stdio.h>
#include <stddef.h>
#include "ptstore.h"
int main(void) {
  printf("%zu %zu %zu %zu %zu %zu\n", sizeof(ptstore_config_t), offsetof(ptstore_config_t, salt), offsetof(ptstore_config_t, table_slots),
         offsetof(ptstore_config_t, device), sizeof(ptstore_paged_cache_t), sizeof(ptstore_stats_t));
  return 0;
}
'''
    with tempfile.TemporaryDirectory() as d:
        path, exe = os.path.join(d, "t.c"), os.path.join(d, "t")
        open(path, "w").write(prog)
        subprocess.check_call(["gcc", "-std=c99", "-I", os.path.join(ROOT, "include"), "-o", exe, path])
        got = [int(x) for x in subprocess.check_output([exe]).split()]
    want = [C.sizeof(Config), Config.salt.offset, Config.table_slots.offset, Config.device.offset, C.sizeof(PagedCache), C.sizeof(Stats)]
    assert got == want


def test_new_entry_points_refuse_bad_arguments_on_the_host():
    """Argument checks that need no device: a null handle, null buffers, sizes out of range."""
    lib = C.CDLL(build.build())
    vp, i32, u32, u64, i64 = C.c_void_p, C.c_int32, C.c_uint32, C.c_uint64, C.c_int64
    lib.ptstore_reserve.argtypes = [vp, i64, i32, vp, i32, u32, vp, vp, i32, vp]
    lib.ptstore_lookup_fetch.argtypes = [vp, vp, vp, i32, i32, u32, vp, vp, vp, vp, vp]
    lib.ptstore_insert_after_lookup.argtypes = [vp, vp, vp, i32, i32, vp, vp, vp, vp, vp]
    lib.ptstore_set_wait_limit.argtypes = [vp, u32]
    lib.ptstore_time_next_copy.argtypes = [vp, vp, vp]
    lib.ptstore_copy_probe.argtypes = [vp, vp, u64, i32, u32, i32, u32, i32, i32, vp, vp]
    lib.ptstore_resumed_inserts.restype = u64
    lib.ptstore_resumed_inserts.argtypes = [vp]
    E_INVAL = -1
    assert lib.ptstore_reserve(None, 10, 0, None, 0, 0, None, None, 0, None) == E_INVAL
    assert lib.ptstore_lookup_fetch(None, None, None, 1, 1, 0, None, None, None, None, None) == E_INVAL
    assert lib.ptstore_insert_after_lookup(None, None, None, 1, 1, None, None, None, None, None) == E_INVAL
    assert lib.ptstore_set_wait_limit(None, 1) == E_INVAL
    assert lib.ptstore_time_next_copy(None, None, None) == E_INVAL
    assert lib.ptstore_resumed_inserts(None) == 0
    # the copy probe checks pointers, alignment, mode, ring geometry and sizes before it touches the device
    a = 1 << 20
    assert lib.ptstore_copy_probe(None, a, 1 << 26, 2, 100, 3, 32768, 1, 0, a, None) == E_INVAL
    assert lib.ptstore_copy_probe(a, a + 8, 1 << 26, 2, 100, 3, 32768, 1, 0, a, None) == E_INVAL          # misaligned
    assert lib.ptstore_copy_probe(a, a, 1 << 26, 7, 100, 3, 32768, 1, 0, a, None) == E_INVAL              # unknown mode
    assert lib.ptstore_copy_probe(a, a, 1 << 26, 2, 100, 1, 32768, 1, 0, a, None) == E_INVAL              # one stage is no ring
    assert lib.ptstore_copy_probe(a, a, 1 << 26, 2, 100, 8, 32768, 1, 0, a, None) == E_INVAL              # ring above 200 KiB
    assert lib.ptstore_copy_probe(a, a, 1 << 26, 3, 50, 3, 32768, 1, 0, a, None) == E_INVAL               # fewer than one store per load
    assert lib.ptstore_copy_probe(a, a, (1 << 26) + 32768, 2, 100, 3, 32768, 1, 0, a, None) == E_INVAL    # not a whole number of units


def build_c_client(out_dir):
    """Compile and link tests/abi_client.c (plain C99) against the library and the CUDA runtime; returns the executable."""
    import subprocess
    lib = build.build()
    cuda = os.environ.get("CUDA_HOME", "/usr/local/cuda")
    exe = os.path.join(out_dir, "abi_client")
    subprocess.check_call(["gcc", "-std=c99", "-Wall", "-Wextra", "-Werror", "-O1", "-I", os.path.join(ROOT, "include"), "-I", os.path.join(cuda, "include"),
                           os.path.join(ROOT, "tests", "abi_client.c"), "-o", exe, lib, "-L", os.path.join(cuda, "lib64"), "-lcudart",
                           "-Wl,-rpath," + os.path.dirname(lib), "-Wl,-rpath," + os.path.join(cuda, "lib64")])
    return exe


def test_a_plain_c_program_compiles_and_links_against_the_library():
    """The boundary is usable from C with nothing but the header, the shared library and the CUDA runtime (the program
    itself runs in the GPU tests)."""
    import tempfile
    with tempfile.TemporaryDirectory() as d:
        assert os.path.exists(build_c_client(d))
