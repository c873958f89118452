"""ctypes binding of the Tetra C-ABI library (include/tetra.h).

Argument marshalling only: every step of the decode-and-multiply path runs in
the CUDA kernels of libtetra_b200.so.  PyTorch supplies device memory and
streams.  There is no CPU fallback: if the library is missing or a call fails,
an exception is raised.
"""
import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("TETRA_LIB") or os.path.join(_HERE, "libtetra_b200.so")

BLOCK = 24
WORD_BYTES = 6
MAX_BATCH = 16
PAPER_TABLE_BYTES = 18816
LIST_MAX = 8


class TetraError(RuntimeError):
    pass


class Q4Problem(C.Structure):
    """Mirror of tetra_q4_problem."""
    _fields_ = [("packed", C.c_void_p), ("x", C.c_void_p), ("y", C.c_void_p), ("N", C.c_int32), ("K", C.c_int32)]


class Problem(C.Structure):
    """Mirror of tetra_problem."""
    _fields_ = [("codes", C.c_void_p), ("row_scales", C.c_void_p), ("x", C.c_void_p),
                ("tail", C.c_void_p), ("y", C.c_void_p), ("N", C.c_int32), ("K", C.c_int32)]


_lib = None


def lib():
    """The loaded library; raises if it has not been built (python -m paper_2609_35465_b200.build)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise TetraError("CUDA library not built: %s is missing (run python -m paper_2609_35465_b200.build)"
                             % LIB_PATH)
        L = C.CDLL(LIB_PATH)
        vp, sz, i32 = C.c_void_p, C.c_size_t, C.c_int
        L.tetra_status_string.argtypes = [i32]
        L.tetra_status_string.restype = C.c_char_p
        L.tetra_table_bytes.argtypes = []
        L.tetra_table_bytes.restype = sz
        L.tetra_build_table.argtypes = [vp, sz, vp, vp]
        L.tetra_table_export.argtypes = [vp, sz]
        L.tetra_decode_blocks.argtypes = [vp, vp, vp, vp, sz, vp]
        L.tetra_codes_bytes.argtypes = [i32, i32]
        L.tetra_codes_bytes.restype = sz
        L.tetra_pack_codes.argtypes = [vp, vp, vp, i32, i32, vp]
        L.tetra_decode_packed.argtypes = [vp, vp, vp, vp, i32, i32, vp]
        L.tetra_gemv.argtypes = [vp, vp, vp, vp, vp, i32, i32, i32, vp]
        L.tetra_gemv_tail.argtypes = [vp, vp, vp, vp, vp, i32, i32, i32, vp, vp]
        L.tetra_gemv_list.argtypes = [vp, i32, vp, vp]
        L.tetra_grouped_workspace_bytes.argtypes = [vp, i32]
        L.tetra_grouped_workspace_bytes.restype = sz
        L.tetra_gemv_grouped_plan.argtypes = [vp, i32, vp, sz, vp]
        L.tetra_gemv_grouped_run.argtypes = [vp, vp, vp]
        L.tetra_gemv_grouped.argtypes = [vp, i32, vp, vp, sz, vp]
        L.tetra_gemv_paper_design.argtypes = [vp, sz, vp, vp, vp, vp, i32, i32, i32, vp, vp]
        L.tetra_gemv_hostio.argtypes = [vp, vp, vp, vp, vp, vp, vp, i32, i32, i32, vp, vp]
        L.tetra_gemv_grouped_hostio.argtypes = [vp, vp, vp, vp, sz, vp, vp, sz, vp]
        L.tetra_batched_workspace_bytes.argtypes = [i32, i32]
        L.tetra_batched_workspace_bytes.restype = sz
        L.tetra_gemv_batched.argtypes = [vp, vp, vp, vp, vp, i32, i32, i32, vp, vp, sz, vp]
        L.tetra_gemv_noalloc.argtypes = [vp, vp, vp, vp, vp, i32, i32, vp, vp]
        L.tetra_encode_blocks.argtypes = [vp, vp, vp, vp, vp, sz, vp]
        L.tetra_q4_packed_bytes.argtypes = [i32, i32, i32]
        L.tetra_q4_packed_bytes.restype = sz
        L.tetra_q4_pack.argtypes = [vp, vp, vp, vp, sz, i32, i32, i32, vp]
        L.tetra_q4_gemv.argtypes = [vp, vp, vp, i32, i32, i32, i32, vp]
        L.tetra_q4_rows.argtypes = [vp, vp, i32, vp, i32, i32, i32, vp]
        L.tetra_q4_list_workspace_bytes.argtypes = [vp, i32, i32]
        L.tetra_q4_list_workspace_bytes.restype = sz
        L.tetra_q4_list_plan.argtypes = [vp, i32, i32, vp, sz, vp]
        L.tetra_q4_list_run.argtypes = [vp, i32, vp]
        _lib = L
    return _lib


def _check(rc: int, what: str):
    if rc != 0:
        raise TetraError("%s failed: %s (%d)" % (what, lib().tetra_status_string(rc).decode(), rc))


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


def _ptr(t):
    return C.c_void_p(t.data_ptr()) if t is not None else C.c_void_p(0)


def _need(t, nbytes: int, what: str, cuda: bool = True):
    """The tensor handed over as `what` holds at least nbytes, contiguously, where the call reads or writes it.
    The C ABI sees plain pointers; a tensor that is too small would be read or written past its end."""
    if t is None:
        return
    have = t.numel() * t.element_size()
    if have < nbytes:
        raise TetraError("%s: tensor of %d bytes, the call needs %d" % (what, have, nbytes))
    if not t.is_contiguous():
        raise TetraError("%s: tensor is not contiguous" % what)
    if cuda and not (t.is_cuda or t.is_pinned()):  # pinned host memory is mapped into the device's address space
        raise TetraError("%s: tensor is neither on the device nor in pinned host memory" % what)


def _blocks(K: int, tail_rule: bool) -> int:
    return K // BLOCK if (tail_rule or K % BLOCK == 0) else -(-K // BLOCK)


def _need_gemv(what, codes, row_scales, x, y, N, K, batch, tail, tail_rule):
    """Sizes of the tensors of one product (tail_rule: floor(K/24) words per row plus a float16 tail)."""
    if N <= 0 or K <= 0 or batch <= 0:
        return  # the library rejects the shape
    B = _blocks(K, tail_rule)
    if B > 0:
        _need(codes, -(-N // 8) * B * 48, what + " codes")
    _need(row_scales, 4 * N, what + " row_scales")
    _need(x, 2 * batch * K, what + " x")
    _need(y, 4 * batch * N, what + " y")
    if tail_rule and K % BLOCK:
        _need(tail, 2 * N * (K % BLOCK), what + " tail")


# ---------------------------------------------------------------------------
def tetra_table_bytes() -> int:
    return lib().tetra_table_bytes()


def tetra_table_export() -> bytes:
    """The paper-format tables (18,816 bytes) as built by the library on the host."""
    buf = C.create_string_buffer(PAPER_TABLE_BYTES)
    _check(lib().tetra_table_export(buf, PAPER_TABLE_BYTES), "tetra_table_export")
    return buf.raw


def tetra_build_table(gain=None, device="cuda", stream=None) -> torch.Tensor:
    """Allocates and fills the device table blob (uint8 tensor)."""
    table = torch.empty(tetra_table_bytes(), dtype=torch.uint8, device=device)
    g = None
    if gain is not None:
        g = (C.c_float * 2)(float(gain[0]), float(gain[1]))
    _check(lib().tetra_build_table(_ptr(table), table.numel(), g, _stream(stream)), "tetra_build_table")
    return table


def tetra_decode_blocks(codes: torch.Tensor, table: torch.Tensor, want_mg: bool = True, stream=None):
    """codes: uint8 [..., 6] file-order words on the device -> (y int8 [n, 24], mg uint8 [n, 2] or None)."""
    assert codes.dtype == torch.uint8 and codes.is_cuda and codes.is_contiguous()
    n = codes.numel() // WORD_BYTES
    y = torch.empty((n, BLOCK), dtype=torch.int8, device=codes.device)
    mg = torch.empty((n, 2), dtype=torch.uint8, device=codes.device) if want_mg else None
    _check(lib().tetra_decode_blocks(_ptr(codes), _ptr(table), _ptr(y), _ptr(mg), n, _stream(stream)),
           "tetra_decode_blocks")
    return y, mg


def tetra_codes_bytes(N: int, nblocks: int) -> int:
    return lib().tetra_codes_bytes(N, nblocks)


def tetra_pack_codes(codes: torch.Tensor, table: torch.Tensor, N: int, nblocks: int, out=None, stream=None):
    """codes: uint8 [N, nblocks, 6] file order on the device -> packed uint8 tensor."""
    assert codes.dtype == torch.uint8 and codes.is_cuda and codes.is_contiguous()
    assert codes.numel() == N * nblocks * WORD_BYTES
    nbytes = tetra_codes_bytes(N, nblocks)
    if out is None:
        out = torch.empty(nbytes, dtype=torch.uint8, device=codes.device)
    assert out.numel() >= nbytes
    _check(lib().tetra_pack_codes(_ptr(codes), _ptr(table), _ptr(out), N, nblocks, _stream(stream)),
           "tetra_pack_codes")
    return out


def tetra_decode_packed(packed: torch.Tensor, table: torch.Tensor, N: int, nblocks: int, want_mg=True, stream=None):
    y = torch.empty((N, nblocks, BLOCK), dtype=torch.int8, device=packed.device)
    mg = torch.empty((N, nblocks, 2), dtype=torch.uint8, device=packed.device) if want_mg else None
    _check(lib().tetra_decode_packed(_ptr(packed), _ptr(table), _ptr(y), _ptr(mg), N, nblocks, _stream(stream)),
           "tetra_decode_packed")
    return y, mg


def tetra_gemv(codes, row_scales, table, x, y, N: int, K: int, batch: int = 1, stream=None):
    """Zero-pad rule: ceil(K/24) words per row."""
    _need_gemv("tetra_gemv", codes, row_scales, x, y, N, K, batch, None, False)
    _check(lib().tetra_gemv(_ptr(codes), _ptr(row_scales), _ptr(table), _ptr(x), _ptr(y), N, K, batch,
                            _stream(stream)), "tetra_gemv")
    return y


def tetra_gemv_tail(codes, row_scales, table, x, y, N: int, K: int, batch: int = 1, tail=None, stream=None):
    """The paper's rule: floor(K/24) words per row plus a float16 tail."""
    _need_gemv("tetra_gemv_tail", codes, row_scales, x, y, N, K, batch, tail, tail is not None)
    _check(lib().tetra_gemv_tail(_ptr(codes), _ptr(row_scales), _ptr(table), _ptr(x), _ptr(y), N, K, batch,
                                 _ptr(tail), _stream(stream)), "tetra_gemv_tail")
    return y


def make_problems(items):
    """items: iterable of dicts(codes, row_scales, x, tail, y, N, K) of device tensors -> ctypes array."""
    items = list(items)
    arr = (Problem * len(items))()
    for i, it in enumerate(items):
        _need_gemv("problem %d" % i, it["codes"], it["row_scales"], it["x"], it["y"], it["N"], it["K"], 1, it.get("tail"),
                   it.get("tail") is not None)
        arr[i] = Problem(it["codes"].data_ptr(), it["row_scales"].data_ptr(), it["x"].data_ptr(),
                         it["tail"].data_ptr() if it.get("tail") is not None else None,
                         it["y"].data_ptr(), it["N"], it["K"])
    return arr


def tetra_gemv_list(problems, table, stream=None):
    """Batch-1 products of a short list (ctypes array from make_problems, at most LIST_MAX) in one launch."""
    _check(lib().tetra_gemv_list(problems, len(problems), _ptr(table), _stream(stream)), "tetra_gemv_list")


def tetra_grouped_workspace_bytes(problems) -> int:
    return lib().tetra_grouped_workspace_bytes(problems, len(problems))


def tetra_gemv_grouped_plan(problems, workspace: torch.Tensor, stream=None):
    """Writes the plan of a list of products (ctypes array from make_problems) into the workspace."""
    _check(lib().tetra_gemv_grouped_plan(problems, len(problems), _ptr(workspace), workspace.numel(),
                                         _stream(stream)), "tetra_gemv_grouped_plan")


def tetra_gemv_grouped_run(workspace: torch.Tensor, table, stream=None):
    """One step of a planned list: activation pre-pass + persistent GEMV kernel."""
    _check(lib().tetra_gemv_grouped_run(_ptr(workspace), _ptr(table), _stream(stream)), "tetra_gemv_grouped_run")


def tetra_gemv_grouped(problems, table, workspace: torch.Tensor, stream=None):
    """plan + run."""
    _check(lib().tetra_gemv_grouped(problems, len(problems), _ptr(table), _ptr(workspace), workspace.numel(),
                                    _stream(stream)), "tetra_gemv_grouped")


def tetra_gemv_paper_design(codes, row_stride: int, row_scales, table, x, y, N: int, K: int, batch: int = 1,
                            tail=None, stream=None):
    _check(lib().tetra_gemv_paper_design(_ptr(codes), row_stride, _ptr(row_scales), _ptr(table), _ptr(x), _ptr(y),
                                         N, K, batch, _ptr(tail), _stream(stream)), "tetra_gemv_paper_design")
    return y


def tetra_gemv_hostio(codes, row_scales, table, x_host, y_host, x_stage, y_stage, N: int, K: int, batch: int = 1,
                      tail=None, stream=None):
    """x_host / y_host: pinned CPU tensors; the copies and the product are enqueued on the stream."""
    _check(lib().tetra_gemv_hostio(_ptr(codes), _ptr(row_scales), _ptr(table), _ptr(x_host), _ptr(y_host),
                                   _ptr(x_stage), _ptr(y_stage), N, K, batch, _ptr(tail), _stream(stream)),
           "tetra_gemv_hostio")


def tetra_gemv_grouped_hostio(workspace, table, x_host, x_dev, y_host=None, y_dev=None, stream=None):
    """A planned run with pinned host activations / results (one copy in, the kernels, one copy out); with
    y_host = y_dev = None the plan's y pointers are taken to aim at mapped pinned host memory (no copy out)."""
    y_bytes = 0 if y_dev is None else y_dev.numel() * y_dev.element_size()
    _check(lib().tetra_gemv_grouped_hostio(_ptr(workspace), _ptr(table), _ptr(x_host), _ptr(x_dev),
                                           x_dev.numel() * x_dev.element_size(), _ptr(y_host), _ptr(y_dev),
                                           y_bytes, _stream(stream)),
           "tetra_gemv_grouped_hostio")


NOALLOC_MAX_K = 24576


def tetra_gemv_noalloc(codes, row_scales, table, x, y, N: int, K: int, tail=None, stream=None):
    """Batch-1 product for callers that may not allocate device memory: the
    scratch buffer lives inside the library (a fixed array, K <= NOALLOC_MAX_K).
    Calls on one device share that array, so they must not overlap on the GPU."""
    _need_gemv("tetra_gemv_noalloc", codes, row_scales, x, y, N, K, 1, tail, tail is not None)
    _check(lib().tetra_gemv_noalloc(_ptr(codes), _ptr(row_scales), _ptr(table), _ptr(x), _ptr(y), N, K,
                                    _ptr(tail), _stream(stream)), "tetra_gemv_noalloc")
    return y


def tetra_batched_workspace_bytes(N: int, K: int) -> int:
    return lib().tetra_batched_workspace_bytes(N, K)


def tetra_gemv_batched(codes, row_scales, table, x, y, N: int, K: int, batch: int, tail=None, workspace=None,
                       stream=None):
    """1..16 activation vectors at once: decode once per block, tensor-core contraction per block."""
    _need_gemv("tetra_gemv_batched", codes, row_scales, x, y, N, K, batch, tail, tail is not None)
    if workspace is None:
        workspace = torch.empty(tetra_batched_workspace_bytes(N, K), dtype=torch.uint8, device=y.device)
    _check(lib().tetra_gemv_batched(_ptr(codes), _ptr(row_scales), _ptr(table), _ptr(x), _ptr(y), N, K, batch,
                                    _ptr(tail), _ptr(workspace), workspace.numel(), _stream(stream)),
           "tetra_gemv_batched")
    return y


# ---------------------------------------------------------------------------
# 4-bit group-quantised matrices (include/tetra_q4.h)
# ---------------------------------------------------------------------------
def tetra_q4_packed_bytes(N: int, K: int, G: int) -> int:
    n = lib().tetra_q4_packed_bytes(N, K, G)
    if n == 0:
        raise TetraError("tetra_q4_packed_bytes: shape rejected (N=%d, K=%d, G=%d)" % (N, K, G))
    return n


def tetra_q4_pack(q, scale, offset, N: int, K: int, G: int, stream=None):
    """File-order matrix (uint8 [N, K/2], float16 [N, K/G] x 2, all on the device) -> packed device buffer."""
    packed = torch.empty(tetra_q4_packed_bytes(N, K, G), dtype=torch.uint8, device=q.device)
    _need(q, N * (K // 2), "tetra_q4_pack q")
    _need(scale, 2 * N * (K // G), "tetra_q4_pack scale")
    _need(offset, 2 * N * (K // G), "tetra_q4_pack offset")
    _check(lib().tetra_q4_pack(_ptr(q), _ptr(scale), _ptr(offset), _ptr(packed), packed.numel(), N, K, G,
                               _stream(stream)), "tetra_q4_pack")
    return packed


def _need_q4(what, packed, x, y, N, K, G, batch):
    n = lib().tetra_q4_packed_bytes(N, K, G)
    if n == 0 or batch <= 0:
        return  # the library rejects the shape
    _need(packed, n, what + " packed")
    _need(x, 2 * batch * K, what + " x")
    _need(y, 4 * batch * N, what + " y")


def tetra_q4_gemv(packed, x, y, N: int, K: int, G: int, batch: int = 1, stream=None):
    _need_q4("tetra_q4_gemv", packed, x, y, N, K, G, batch)
    _check(lib().tetra_q4_gemv(_ptr(packed), _ptr(x), _ptr(y), N, K, G, batch, _stream(stream)), "tetra_q4_gemv")
    return y


def tetra_q4_rows(packed, ids, out, N: int, K: int, G: int, stream=None):
    _need_q4("tetra_q4_rows", packed, None, None, N, K, G, 1)
    _need(ids, 4 * int(ids.numel()), "tetra_q4_rows ids")
    _need(out, 2 * int(ids.numel()) * K, "tetra_q4_rows out")
    _check(lib().tetra_q4_rows(_ptr(packed), _ptr(ids), int(ids.numel()), _ptr(out), N, K, G, _stream(stream)),
           "tetra_q4_rows")
    return out


def tetra_encode_blocks(w, table, sigma=None, want_cosine=True, stream=None):
    """w: float32 [n, 24] on the device -> (codes uint8 [n, 6] in file order, cosines float32 [n] or None)."""
    n = w.numel() // 24
    _need(w, 4 * 24 * n, "tetra_encode_blocks w")
    _need(sigma, 4 * n, "tetra_encode_blocks sigma")
    codes = torch.empty((n, 6), dtype=torch.uint8, device=w.device)
    cos = torch.empty(n, dtype=torch.float32, device=w.device) if want_cosine else None
    _check(lib().tetra_encode_blocks(_ptr(w), _ptr(sigma), _ptr(table), _ptr(codes), _ptr(cos), n, _stream(stream)),
           "tetra_encode_blocks")
    return codes, cos


def make_q4_problems(items):
    """items: iterable of dicts(packed, x, y, N, K) of device tensors -> ctypes array of tetra_q4_problem."""
    items = list(items)
    arr = (Q4Problem * len(items))()
    for i, it in enumerate(items):
        arr[i] = Q4Problem(it["packed"].data_ptr(), it["x"].data_ptr(), it["y"].data_ptr(), it["N"], it["K"])
    return arr


def tetra_q4_list_plan(problems, G: int, stream=None) -> torch.Tensor:
    """Plans a list of 4-bit products (one group size); returns the workspace tensor to pass to the run."""
    n = lib().tetra_q4_list_workspace_bytes(problems, len(problems), G)
    if n == 0:
        raise TetraError("tetra_q4_list_workspace_bytes: list rejected")
    ws = torch.empty(n, dtype=torch.uint8, device="cuda")
    _check(lib().tetra_q4_list_plan(problems, len(problems), G, _ptr(ws), ws.numel(), _stream(stream)),
           "tetra_q4_list_plan")
    return ws


def tetra_q4_list_run(workspace: torch.Tensor, G: int, stream=None):
    _check(lib().tetra_q4_list_run(_ptr(workspace), G, _stream(stream)), "tetra_q4_list_run")
