"""The C-ABI library builds, loads without a GPU and exports every function the headers under include/ declare.
No compute call is made here."""
import ctypes
import os
import re

from paper_2311_00368_b200 import build as b2sp_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    names = set()
    inc = os.path.join(ROOT, "include")
    for header in sorted(os.listdir(inc)):
        if header.endswith(".h"):
            text = open(os.path.join(inc, header)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\b(b2sp_[a-z0-9_]+)\s*\(", text))
    return sorted(names)


def test_header_declares_the_three_ops():
    names = declared_functions()
    for n in ("b2sp_spmm", "b2sp_sddmm", "b2sp_fusedmm", "b2sp_workspace_bytes", "b2sp_spmm_host",
              "b2sp_sddmm_host", "b2sp_fusedmm_host"):
        assert n in names


def test_library_exports_every_declared_symbol():
    lib = ctypes.CDLL(b2sp_build.build())
    for name in declared_functions():
        assert hasattr(lib, name), f"{name} is declared under include/ but not exported"
    lib.b2sp_version.restype = ctypes.c_int
    assert lib.b2sp_version() >= 100
    lib.b2sp_status_string.restype = ctypes.c_char_p
    assert lib.b2sp_status_string(0) == b"ok"
    lib.b2sp_workspace_bytes.restype = ctypes.c_size_t
    lib.b2sp_workspace_bytes.argtypes = [ctypes.c_int] * 5 + [ctypes.c_longlong]
    n = lib.b2sp_workspace_bytes(2, 8192, 8192, 128, 512, 20_000_000)
    assert n >= 4 * 8192 and n % 256 == 0
    assert lib.b2sp_workspace_bytes(7, 1, 1, 1, 1, 1) == 0
    # per-algo sizes: the row family needs a few bytes per row, the dense-tile family the window table
    # and operand copies; AUTO reports what it would use; the general query bounds them all
    lib.b2sp_workspace_bytes_algo.restype = ctypes.c_size_t
    lib.b2sp_workspace_bytes_algo.argtypes = [ctypes.c_int] * 6 + [ctypes.c_longlong]
    dims = (8192, 8192, 128, 512, 20_000_000)
    row, tile, auto = (lib.b2sp_workspace_bytes_algo(2, a, *dims) for a in (1, 3, 0))
    assert 4 * 8192 <= row < 1 << 20 and tile > 8 * 8192 * 256 and auto == tile == n
    sparse = (8192, 8192, 128, 512, 100_000)     # 0.15% density: AUTO stays with the row family
    assert lib.b2sp_workspace_bytes_algo(2, 0, *sparse) == lib.b2sp_workspace_bytes_algo(2, 1, *sparse)
    assert lib.b2sp_workspace_bytes(2, *sparse) >= lib.b2sp_workspace_bytes_algo(2, 3, *sparse) > 0
    assert lib.b2sp_workspace_bytes_algo(2, 3, 64, 64, 200, 64, 100) == 0   # Kd > 128: outside the tile family
    assert lib.b2sp_workspace_bytes_algo(2, 9, *dims) == 0


def test_argument_errors_need_no_gpu():
    """Argument checks run before any CUDA call."""
    lib = ctypes.CDLL(b2sp_build.build())
    i, ll, vp, sz = ctypes.c_int, ctypes.c_longlong, ctypes.c_void_p, ctypes.c_size_t
    lib.b2sp_spmm.restype = i
    lib.b2sp_spmm.argtypes = [i, i, i, ll, vp, vp, vp, vp, ll, vp, ll, vp, sz, i, vp]
    assert lib.b2sp_spmm(-1, 4, 4, 0, None, None, None, None, 4, None, 4, None, 0, 0, None) == 1
    assert lib.b2sp_spmm(4, 4, 4, 2 ** 31, None, None, None, None, 4, None, 4, None, 0, 0, None) == 1
    assert lib.b2sp_spmm(4, 4, 4, 3, None, None, None, None, 4, None, 4, None, 0, 0, None) == 1


def test_binding_refuses_to_run_without_the_library(tmp_path, monkeypatch):
    """There is no fallback: without libb2sp.so the binding cannot even be imported."""
    import importlib.util
    src = os.path.join(ROOT, "paper_2311_00368_b200", "binding.py")
    dst = tmp_path / "binding_copy.py"
    dst.write_text(open(src).read())
    spec = importlib.util.spec_from_file_location("binding_copy", dst)
    mod = importlib.util.module_from_spec(spec)
    try:
        spec.loader.exec_module(mod)
        raised = False
    except ImportError:
        raised = True
    assert raised


def test_batched_and_bf16_entry_points_check_arguments_without_a_gpu():
    lib = ctypes.CDLL(b2sp_build.build())
    i, ll, vp, sz = ctypes.c_int, ctypes.c_longlong, ctypes.c_void_p, ctypes.c_size_t
    lib.b2sp_workspace_bytes_batched.restype = sz
    lib.b2sp_workspace_bytes_batched.argtypes = [i, i, i, i, i, ll]
    one = lib.b2sp_workspace_bytes_batched(1, 4096, 4096, 64, 64, 3_400_000)
    eight = lib.b2sp_workspace_bytes_batched(8, 4096, 4096, 64, 64, 3_400_000)
    assert one % 256 == 0 and eight > 4 * one > 0            # tables and operand copies are per problem (a single problem also holds K-split slabs)
    assert lib.b2sp_workspace_bytes_batched(0, 4096, 4096, 64, 64, 3_400_000) == 0
    wide = lib.b2sp_workspace_bytes_batched(8, 4096, 4096, 64, 512, 3_400_000)
    assert 0 < wide < 1 << 20                                # wider than 256 columns: the row kernels' few bytes per row
    lib.b2sp_fusedmm_batched.restype = i
    lib.b2sp_fusedmm_batched.argtypes = [i, i, i, i, i, ll, vp, ll, vp, vp, vp, ll, ll, vp, ll, ll, vp, ll, ll, vp, ll, ll,
                                         vp, sz, i, vp]
    args = [2, 64, 64, 16, 16, 100, None, 65, None, None, None, 16, 1024, None, 16, 1024, None, 16, 1024, None, 16, 1024,
            None, 0, 0, None]
    assert lib.b2sp_fusedmm_batched(*args) == 1              # NULL row_ptr
    args[0] = 0
    assert lib.b2sp_fusedmm_batched(*args) == 1              # empty batch
    lib.b2sp_spmm_bf16.restype = i
    lib.b2sp_spmm_bf16.argtypes = [i, i, i, ll, vp, vp, vp, vp, ll, vp, ll, vp, sz, i, vp]
    assert lib.b2sp_spmm_bf16(-1, 4, 4, 0, None, None, None, None, 4, None, 4, None, 0, 0, None) == 1
    assert lib.b2sp_spmm_bf16(4, 4, 4, 3, None, None, None, None, 4, None, 4, None, 0, 0, None) == 1
