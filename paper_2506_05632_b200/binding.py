"""ctypes binding of libgls.so (C ABI in include/gls.h).  Argument marshalling only."""
import ctypes as C
import os
import subprocess
import threading

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_HERE)
_SRC_DIR = os.path.join(_HERE, "csrc")
_LIB = os.path.join(_HERE, "libgls.so")

COMBINE_ACTIVE, COMBINE_ALL, NO_BONUS = 0, 1, 2
VERIFY_ALL_ROWS, VERIFY_ACTIVE_ROWS = 4, 8  # how the dense verify call walks Algorithm 2
VERIFY_FIRST_PHASE, VERIFY_REST = 16, 32   # the walk in phases as two calls (rows fetched on demand)
VERIFY_THREE_PHASES = 64                   # positions 1 and 2 as a phase of their own
NOISE_SHARED_ACROSS_K = 1
DEV_EMPTY_SUPPORT = 1
F32, BF16 = 0, 1

_lock = threading.Lock()
_lib = None


class GlsError(RuntimeError):
    pass


def lib_path():
    return _LIB


def _sources():
    return sorted(os.path.join(_SRC_DIR, f) for f in os.listdir(_SRC_DIR)
                  if f.endswith((".cu", ".cuh"))) + [os.path.join(_ROOT, "include", "gls.h")]


def build(force=False, verbose=False, debug_bounds=False):
    """Compile csrc/*.cu into libgls.so for sm_100a with nvcc (cross-compiles without a GPU)."""
    srcs = _sources()
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= max(os.path.getmtime(s) for s in srcs)):
        return _LIB
    cus = [s for s in srcs if s.endswith(".cu")]
    tmp = _LIB + ".tmp%d" % os.getpid()
    cmd = ["nvcc", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-shared", "-Xcompiler", "-fPIC", "-o", tmp] + cus
    if debug_bounds or os.environ.get("GLS_DEBUG_BOUNDS") == "1":
        cmd.insert(1, "-DGLS_DEBUG_BOUNDS")  # range checks of the kernels' own indices
    if verbose:
        cmd.insert(1, "-Xptxas=-v")
    subprocess.run(cmd, check=True)
    os.replace(tmp, _LIB)
    return _LIB


class _Rows(C.Structure):
    _fields_ = [("data", C.c_void_p), ("dtype", C.c_int32), ("stride_b", C.c_int64),
                ("stride_k", C.c_int64), ("stride_j", C.c_int64)]


class _SparseRows(C.Structure):
    _fields_ = [("token_ids", C.c_void_p), ("logits", C.c_void_p), ("stride_b", C.c_int64),
                ("stride_k", C.c_int64), ("stride_j", C.c_int64), ("M", C.c_int32)]


class _Noise(C.Structure):
    _fields_ = [("seed", C.c_uint64), ("seq_base", C.c_uint32), ("seq_ids", C.c_void_p),
                ("pos_base", C.c_uint32), ("noise_spec", C.c_uint32), ("rounds", C.c_uint32),
                ("flags", C.c_uint32)]


def load():
    """Load libgls.so (building it if the sources are newer and nvcc is present)."""
    global _lib
    with _lock:
        if _lib is not None:
            return _lib
        if not os.path.exists(_LIB):
            build()
        L = C.CDLL(_LIB)
        L.gls_version.restype = C.c_int
        L.gls_status_string.restype = C.c_char_p
        L.gls_status_string.argtypes = [C.c_int]
        L.gls_workspace_bytes.restype = C.c_size_t
        L.gls_workspace_bytes.argtypes = [C.c_int, C.c_int, C.c_int, C.c_int64]
        L.gls_draft_sample.restype = C.c_int
        L.gls_draft_sample.argtypes = [
            C.POINTER(_Rows), C.c_int, C.c_int, C.c_int, C.c_int64, C.c_float, C.c_void_p,
            C.POINTER(_Noise), C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p,
            C.c_void_p]
        L.gls_static_scratch_bytes.restype = C.c_size_t
        L.gls_draft_sample_static.restype = C.c_int
        L.gls_draft_sample_static.argtypes = [
            C.POINTER(_Rows), C.c_int, C.c_int, C.c_int, C.c_int64, C.c_float, C.c_void_p,
            C.POINTER(_Noise), C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.gls_draft_sample_sparse.restype = C.c_int
        L.gls_draft_sample_sparse.argtypes = [
            C.POINTER(_SparseRows), C.c_int, C.c_int, C.c_int, C.c_float, C.c_void_p,
            C.POINTER(_Noise), C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.gls_target_sample_verify_sparse.restype = C.c_int
        L.gls_target_sample_verify_sparse.argtypes = [
            C.POINTER(_SparseRows), C.c_int, C.c_int, C.c_int, C.c_float, C.c_void_p,
            C.POINTER(_Noise), C.c_uint32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
            C.c_void_p, C.c_void_p]
        L.gls_target_sample_verify.restype = C.c_int
        L.gls_target_sample_verify.argtypes = [
            C.POINTER(_Rows), C.c_int, C.c_int, C.c_int, C.c_int64, C.c_float, C.c_void_p,
            C.POINTER(_Noise), C.c_uint32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
            C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p]
        L.gls_draft_verify_workspace_bytes.restype = C.c_size_t
        L.gls_draft_verify_workspace_bytes.argtypes = [C.c_int, C.c_int, C.c_int, C.c_int, C.c_int64]
        L.gls_draft_verify.restype = C.c_int
        L.gls_draft_verify.argtypes = [
            C.POINTER(_Rows), C.POINTER(_Rows), C.c_int, C.c_int, C.c_int, C.c_int64, C.c_float,
            C.c_void_p, C.c_float, C.POINTER(_Noise), C.c_uint32, C.c_void_p, C.c_void_p, C.c_void_p,
            C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p]
        L.gls_topm_workspace_bytes.restype = C.c_size_t
        L.gls_topm_workspace_bytes.argtypes = [C.c_int, C.c_int, C.c_int, C.c_int]
        L.gls_draft_sample_topm.restype = C.c_int
        L.gls_draft_sample_topm.argtypes = [
            C.POINTER(_Rows), C.c_int, C.c_int, C.c_int, C.c_int64, C.c_int, C.c_float, C.c_void_p,
            C.POINTER(_Noise), C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p,
            C.c_void_p]
        L.gls_target_sample_verify_topm.restype = C.c_int
        L.gls_target_sample_verify_topm.argtypes = [
            C.POINTER(_Rows), C.c_int, C.c_int, C.c_int, C.c_int64, C.c_int, C.c_float, C.c_void_p,
            C.POINTER(_Noise), C.c_uint32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
            C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p]
        L.gls_compress_gaussian_workspace_bytes.restype = C.c_size_t
        L.gls_compress_gaussian_workspace_bytes.argtypes = [C.c_int, C.c_int, C.c_int64]
        L.gls_compress_gaussian.restype = C.c_int
        L.gls_compress_gaussian.argtypes = [
            C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_int, C.c_int, C.c_int64,
            C.c_int, C.c_double, C.c_double, C.c_double, C.POINTER(_Noise), C.c_void_p, C.c_void_p,
            C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t,
            C.c_void_p, C.c_void_p]
        L.gls_compress_select.restype = C.c_int
        L.gls_compress_select.argtypes = [
            C.POINTER(_Rows), C.POINTER(_Rows), C.c_void_p, C.c_int64, C.c_int, C.c_int,
            C.c_int64, C.POINTER(_Noise), C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
            C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p]
        _lib = L
        return _lib


def debug_bounds():
    """(compiled in?, [count, first site, value, limit]) of the library's index self-check."""
    out = (C.c_uint32 * 4)()
    L = load()
    L.gls_debug_bounds.restype = C.c_int
    rc = int(L.gls_debug_bounds(out))
    return rc, [int(x) for x in out]


def version():
    return int(load().gls_version())


def status_string(rc):
    return load().gls_status_string(int(rc)).decode()


def workspace_bytes(B, K, J, V):
    return int(load().gls_workspace_bytes(int(B), int(K), int(J), int(V)))


def _check(rc):
    if rc != 0:
        raise GlsError(status_string(rc))


def _rows(t, lead):
    """gls_rows_t of a tensor whose last dim is contiguous; `lead` leading dims give strides."""
    if not t.is_cuda:
        raise GlsError("libgls takes device tensors; there is no CPU path")
    if t.dtype == torch.float32:
        dt = F32
    elif t.dtype == torch.bfloat16:
        dt = BF16
    else:
        raise GlsError("logits must be float32 or bfloat16")
    if t.stride(-1) != 1 and t.shape[-1] > 1:
        raise GlsError("the token dimension must be contiguous")
    st = [t.stride(d) for d in range(lead)] + [0] * (3 - lead)
    return _Rows(t.data_ptr(), dt, st[0], st[1], st[2])


def _noise(seed, seq_base, seq_ids, pos_base, spec, rounds, flags):
    ptr = None
    if seq_ids is not None:
        if seq_ids.dtype != torch.int32 or not seq_ids.is_cuda or not seq_ids.is_contiguous():
            raise GlsError("seq_ids must be a contiguous int32 device tensor (bit pattern = uint32)")
        ptr = seq_ids.data_ptr()
    return _Noise(int(seed) & (2**64 - 1), int(seq_base), ptr, int(pos_base), int(spec),
                  int(rounds), int(flags))


def _ptr(t):
    return None if t is None else t.data_ptr()


def _stream():
    return torch.cuda.current_stream().cuda_stream


def _workspace(workspace, need, device):
    if workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device=device)
    return workspace


def draft_sample(logits, inv_temp=1.0, inv_temp_per_draft=None, seed=0, seq_base=0, seq_ids=None,
                 pos_base=0, spec=4, rounds=10, noise_flags=0, want_scores=True, workspace=None,
                 status=None, out_tokens=None, out_scores=None):
    """logits [B,K,J,V] (device, fp32/bf16) -> (tokens int32 [B,K,J], scores fp32 [B,K,J] | None)."""
    L = load()
    B, K, J, V = logits.shape
    dev = logits.device
    rows = _rows(logits, 3)
    nz = _noise(seed, seq_base, seq_ids, pos_base, spec, rounds, noise_flags)
    if out_tokens is None:
        out_tokens = torch.empty((B, K, J), dtype=torch.int32, device=dev)
    if out_scores is None and want_scores:
        out_scores = torch.empty((B, K, J), dtype=torch.float32, device=dev)
    need = workspace_bytes(B, K, J, V)
    workspace = _workspace(workspace, need, dev)
    itk = None
    if inv_temp_per_draft is not None:
        itk = (C.c_float * K)(*[float(x) for x in inv_temp_per_draft])
    _check(L.gls_draft_sample(C.byref(rows), B, K, J, V, float(inv_temp),
                              C.cast(itk, C.c_void_p) if itk is not None else None, C.byref(nz),
                              _ptr(out_tokens), _ptr(out_scores), workspace.data_ptr(),
                              workspace.numel(), _ptr(status), _stream()))
    return out_tokens, out_scores


def static_scratch_bytes():
    return int(load().gls_static_scratch_bytes())


def draft_sample_static(logits, out_tokens, out_scores=None, inv_temp=1.0, inv_temp_per_draft=None,
                        seed=0, seq_base=0, seq_ids=None, pos_base=0, spec=4, rounds=10,
                        noise_flags=0, status=None):
    """gls_draft_sample_static: draft_sample for callers that may not allocate device memory.

    The caller passes the outputs (int32 [B,K,J], optional fp32 [B,K,J]); this wrapper creates no
    tensor and the library uses its built-in scratch buffer.  Raises GlsError when the problem
    needs more scratch than static_scratch_bytes()."""
    L = load()
    B, K, J, V = logits.shape
    rows = _rows(logits, 3)
    nz = _noise(seed, seq_base, seq_ids, pos_base, spec, rounds, noise_flags)
    itk = None
    if inv_temp_per_draft is not None:
        itk = (C.c_float * K)(*[float(x) for x in inv_temp_per_draft])
    _check(L.gls_draft_sample_static(C.byref(rows), B, K, J, V, float(inv_temp),
                                     C.cast(itk, C.c_void_p) if itk is not None else None,
                                     C.byref(nz), _ptr(out_tokens), _ptr(out_scores), _ptr(status),
                                     _stream()))
    return out_tokens, out_scores


def _sparse(ids, logits):
    """gls_sparse_rows_t of ids int32 [B,K,J,M] and logits fp32 with the same shape and strides."""
    if not (ids.is_cuda and logits.is_cuda):
        raise GlsError("libgls takes device tensors; there is no CPU path")
    if ids.dtype != torch.int32 or logits.dtype != torch.float32:
        raise GlsError("sparse rows are int32 token ids and float32 logits")
    if ids.shape != logits.shape or ids.stride() != logits.stride():
        raise GlsError("token_ids and logits must share shape and strides")
    if ids.stride(-1) != 1 and ids.shape[-1] > 1:
        raise GlsError("the kept-token dimension must be contiguous")
    return _SparseRows(ids.data_ptr(), logits.data_ptr(), ids.stride(0), ids.stride(1),
                       ids.stride(2), ids.shape[3])


def draft_sample_sparse(token_ids, logits, inv_temp=1.0, inv_temp_per_draft=None, seed=0,
                        seq_base=0, seq_ids=None, pos_base=0, spec=4, rounds=10, noise_flags=0,
                        want_scores=True, status=None):
    """Sparse rows (kept token ids and their logits, [B,K,J,M]) -> (vocabulary ids int32 [B,K,J],
    scores fp32 [B,K,J] | None).  Same races as draft_sample on the row masked to the kept tokens."""
    L = load()
    B, K, J, M = token_ids.shape
    rows = _sparse(token_ids, logits)
    nz = _noise(seed, seq_base, seq_ids, pos_base, spec, rounds, noise_flags)
    dev = token_ids.device
    out_tokens = torch.empty((B, K, J), dtype=torch.int32, device=dev)
    out_scores = torch.empty((B, K, J), dtype=torch.float32, device=dev) if want_scores else None
    itk = None
    if inv_temp_per_draft is not None:
        itk = (C.c_float * K)(*[float(x) for x in inv_temp_per_draft])
    _check(L.gls_draft_sample_sparse(C.byref(rows), B, K, J, float(inv_temp),
                                     C.cast(itk, C.c_void_p) if itk is not None else None,
                                     C.byref(nz), _ptr(out_tokens), _ptr(out_scores), _ptr(status),
                                     _stream()))
    return out_tokens, out_scores


def target_sample_verify_sparse(token_ids, logits, draft_tokens, inv_temp=1.0, flags=0, seed=0,
                                seq_base=0, seq_ids=None, pos_base=0, spec=4, rounds=10,
                                noise_flags=0, want_scores=True, status=None):
    """Sparse target rows [B,K,J,M] (J = L+1, or L with NO_BONUS) and draft_tokens int32 [B,K,L]
    -> dict(tokens [B,J], tau [B], accept [B,K,L], scores [B,J] | None)."""
    L = load()
    B, K, J, M = token_ids.shape
    Ld = J if (flags & NO_BONUS) else J - 1
    rows = _sparse(token_ids, logits)
    nz = _noise(seed, seq_base, seq_ids, pos_base, spec, rounds, noise_flags)
    dev = token_ids.device
    if Ld > 0:
        if draft_tokens.dtype != torch.int32 or not draft_tokens.is_contiguous():
            raise GlsError("draft_tokens must be contiguous int32")
        assert tuple(draft_tokens.shape) == (B, K, Ld)
    out = dict(tokens=torch.empty((B, J), dtype=torch.int32, device=dev),
               tau=torch.empty((B,), dtype=torch.int32, device=dev),
               accept=torch.empty((B, K, Ld), dtype=torch.uint8, device=dev),
               scores=torch.empty((B, J), dtype=torch.float32, device=dev) if want_scores else None)
    _check(L.gls_target_sample_verify_sparse(
        C.byref(rows), B, K, Ld, float(inv_temp), _ptr(draft_tokens) if Ld > 0 else None,
        C.byref(nz), int(flags), _ptr(out["tokens"]), _ptr(out["tau"]),
        _ptr(out["accept"]) if Ld > 0 else None, _ptr(out.get("scores")), _ptr(status), _stream()))
    return out


def topm_workspace_bytes(B, K, J, M):
    return int(load().gls_topm_workspace_bytes(int(B), int(K), int(J), int(M)))


def _topm_lists(workspace, B, K, J, M):
    """Views of the kept (ids int32, logits fp32) lists [B,K,J,M] a top-M call left in its workspace."""
    n = B * K * J * M
    off = (n * 4 + 255) // 256 * 256
    ids = workspace[:n * 4].view(torch.int32).view(B, K, J, M)
    lg = workspace[off:off + n * 4].view(torch.float32).view(B, K, J, M)
    return ids, lg


def draft_sample_topm(logits, M, inv_temp=1.0, inv_temp_per_draft=None, seed=0, seq_base=0,
                      seq_ids=None, pos_base=0, spec=4, rounds=10, noise_flags=0, want_scores=True,
                      workspace=None, status=None):
    """Dense logits [B,K,J,V] truncated to their M largest per row, then draft_sample_sparse.

    Returns (tokens int32 [B,K,J], scores | None, (kept ids, kept logits) views [B,K,J,M])."""
    L = load()
    B, K, J, V = logits.shape
    dev = logits.device
    rows = _rows(logits, 3)
    nz = _noise(seed, seq_base, seq_ids, pos_base, spec, rounds, noise_flags)
    out_tokens = torch.empty((B, K, J), dtype=torch.int32, device=dev)
    out_scores = torch.empty((B, K, J), dtype=torch.float32, device=dev) if want_scores else None
    workspace = _workspace(workspace, topm_workspace_bytes(B, K, J, M), dev)
    itk = None
    if inv_temp_per_draft is not None:
        itk = (C.c_float * K)(*[float(x) for x in inv_temp_per_draft])
    _check(L.gls_draft_sample_topm(C.byref(rows), B, K, J, V, int(M), float(inv_temp),
                                   C.cast(itk, C.c_void_p) if itk is not None else None,
                                   C.byref(nz), _ptr(out_tokens), _ptr(out_scores),
                                   workspace.data_ptr(), workspace.numel(), _ptr(status), _stream()))
    return out_tokens, out_scores, _topm_lists(workspace, B, K, J, M)


def target_sample_verify_topm(logits, draft_tokens, M, inv_temp=1.0, flags=0, seed=0, seq_base=0,
                              seq_ids=None, pos_base=0, spec=4, rounds=10, noise_flags=0,
                              want_scores=True, workspace=None, status=None):
    """Dense target logits [B,K,J,V] truncated to their M largest per row, then
    target_sample_verify_sparse.  Returns dict(tokens, tau, accept, scores | None)."""
    L = load()
    B, K, J, V = logits.shape
    Ld = J if (flags & NO_BONUS) else J - 1
    dev = logits.device
    rows = _rows(logits, 3)
    nz = _noise(seed, seq_base, seq_ids, pos_base, spec, rounds, noise_flags)
    if Ld > 0:
        if draft_tokens.dtype != torch.int32 or not draft_tokens.is_contiguous():
            raise GlsError("draft_tokens must be contiguous int32")
        assert tuple(draft_tokens.shape) == (B, K, Ld)
    out = dict(tokens=torch.empty((B, J), dtype=torch.int32, device=dev),
               tau=torch.empty((B,), dtype=torch.int32, device=dev),
               accept=torch.empty((B, K, Ld), dtype=torch.uint8, device=dev),
               scores=torch.empty((B, J), dtype=torch.float32, device=dev) if want_scores else None)
    workspace = _workspace(workspace, topm_workspace_bytes(B, K, J, M), dev)
    _check(L.gls_target_sample_verify_topm(
        C.byref(rows), B, K, Ld, V, int(M), float(inv_temp),
        _ptr(draft_tokens) if Ld > 0 else None, C.byref(nz), int(flags), _ptr(out["tokens"]),
        _ptr(out["tau"]), _ptr(out["accept"]) if Ld > 0 else None, _ptr(out.get("scores")),
        workspace.data_ptr(), workspace.numel(), _ptr(status), _stream()))
    return out


def target_sample_verify(logits, draft_tokens, inv_temp=1.0, flags=0, seed=0, seq_base=0,
                         seq_ids=None, pos_base=0, spec=4, rounds=10, noise_flags=0,
                         want_scores=True, workspace=None, status=None, out=None):
    """logits [B,K,J,V], draft_tokens int32 [B,K,L]; J = L+1 (L with NO_BONUS).

    Returns dict(tokens [B,J], tau [B], accept [B,K,L], scores [B,J] | None)."""
    L = load()
    B, K, J, V = logits.shape
    Ld = J if (flags & NO_BONUS) else J - 1
    dev = logits.device
    rows = _rows(logits, 3)
    nz = _noise(seed, seq_base, seq_ids, pos_base, spec, rounds, noise_flags)
    if Ld > 0:
        if draft_tokens.dtype != torch.int32 or not draft_tokens.is_contiguous():
            raise GlsError("draft_tokens must be contiguous int32")
        assert tuple(draft_tokens.shape) == (B, K, Ld)
    if out is None:
        out = dict(tokens=torch.empty((B, J), dtype=torch.int32, device=dev),
                   tau=torch.empty((B,), dtype=torch.int32, device=dev),
                   accept=torch.empty((B, K, Ld), dtype=torch.uint8, device=dev),
                   scores=torch.empty((B, J), dtype=torch.float32, device=dev)
                   if want_scores else None)
    need = workspace_bytes(B, K, J, V)
    workspace = _workspace(workspace, need, dev)
    _check(L.gls_target_sample_verify(
        C.byref(rows), B, K, Ld, V, float(inv_temp), _ptr(draft_tokens) if Ld > 0 else None,
        C.byref(nz), int(flags), _ptr(out["tokens"]), _ptr(out["tau"]),
        _ptr(out["accept"]) if Ld > 0 else None, _ptr(out.get("scores")), workspace.data_ptr(),
        workspace.numel(), _ptr(status), _stream()))
    return out


def copy_rows_to_device(dst, src, stream=None):
    """dst (device) and src (pinned host): tensors of the same shape [n, row] and dtype whose rows
    are contiguous and a constant stride apart (e.g. t[:, :, 0].flatten(0, 1) of a [B,K,J,V]
    tensor): one strided host-to-device copy on `stream` (default: the current stream)."""
    assert dst.dim() == 2 and dst.shape == src.shape and dst.dtype == src.dtype
    assert dst.is_cuda and not src.is_cuda
    if dst.shape[1] > 1 and (dst.stride(1) != 1 or src.stride(1) != 1):
        raise GlsError("rows must be contiguous")
    es = dst.element_size()
    lib = load()
    lib.gls_copy_rows_to_device.restype = C.c_int
    lib.gls_copy_rows_to_device.argtypes = [C.c_void_p, C.c_size_t, C.c_void_p, C.c_size_t, C.c_size_t,
                                            C.c_size_t, C.c_void_p]
    n, row = dst.shape
    st = stream.cuda_stream if stream is not None else _stream()
    _check(lib.gls_copy_rows_to_device(dst.data_ptr(), max(dst.stride(0), row) * es, src.data_ptr(),
                                       max(src.stride(0), row) * es, row * es, n, st))


def verify_walk(target_logits, L, flags=0, spec=4):
    """1 if target_sample_verify would walk Algorithm 2 in phases for these rows (reading the rows
    of active drafts only), 0 if it would race every row first; GlsError for refused arguments."""
    B, K, J, V = target_logits.shape
    lib = load()
    lib.gls_verify_walk.restype = C.c_int
    lib.gls_verify_walk.argtypes = [C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int64, C.c_int,
                                    C.c_uint32]
    rc = int(lib.gls_verify_walk(BF16 if target_logits.dtype == torch.bfloat16 else F32,
                                 int(target_logits.stride(1) != 0), B, K, int(L), V, int(spec), int(flags)))
    if rc < 0:
        raise GlsError("gls_verify_walk: arguments that the verify call refuses")
    return rc


def verify_phases(target_logits, L, flags=0, spec=4):
    """Phase boundaries of target_sample_verify's walk for these rows: [] if every row is raced,
    else [e0, e1, ...] with phase p covering positions [e(p-1), ep)."""
    B, K, J, V = target_logits.shape
    lib = load()
    ends = (C.c_int * 4)()
    lib.gls_verify_phases.restype = C.c_int
    lib.gls_verify_phases.argtypes = [C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int64, C.c_int,
                                      C.c_uint32, C.c_void_p]
    n = int(lib.gls_verify_phases(BF16 if target_logits.dtype == torch.bfloat16 else F32,
                                  int(target_logits.stride(1) != 0), B, K, int(L), V, int(spec),
                                  int(flags), ends))
    if n < 0:
        raise GlsError("gls_verify_phases: arguments that the verify call refuses")
    return [int(ends[i]) for i in range(n)]


def draft_verify_workspace_bytes(B, K, L, J, V):
    return int(load().gls_draft_verify_workspace_bytes(int(B), int(K), int(L), int(J), int(V)))


def draft_verify(draft_logits, target_logits, inv_temp=1.0, inv_temp_per_draft=None,
                 inv_temp_target=None, flags=0, seed=0, seq_base=0, seq_ids=None, pos_base=0,
                 spec=4, rounds=10, noise_flags=0, want_scores=True, workspace=None, status=None,
                 out_draft_tokens=None, out_draft_scores=None, out=None):
    """gls_draft_verify: draft_logits [B,K,L,V] and target_logits [B,K,J,V] (J = L+1, or L with
    NO_BONUS) in one call.  Returns (draft tokens [B,K,L], draft scores | None, dict(tokens, tau,
    accept, scores | None)) -- what draft_sample followed by target_sample_verify return."""
    L_ = load()
    B, K, L, V = draft_logits.shape
    J = target_logits.shape[2]
    assert tuple(target_logits.shape) == (B, K, J, V) and J == (L if (flags & NO_BONUS) else L + 1)
    dev = draft_logits.device
    drows, trows = _rows(draft_logits, 3), _rows(target_logits, 3)
    nz = _noise(seed, seq_base, seq_ids, pos_base, spec, rounds, noise_flags)
    if out_draft_tokens is None:
        out_draft_tokens = torch.empty((B, K, L), dtype=torch.int32, device=dev)
    if out_draft_scores is None and want_scores:
        out_draft_scores = torch.empty((B, K, L), dtype=torch.float32, device=dev)
    if out is None:
        out = dict(tokens=torch.empty((B, J), dtype=torch.int32, device=dev),
                   tau=torch.empty((B,), dtype=torch.int32, device=dev),
                   accept=torch.empty((B, K, L), dtype=torch.uint8, device=dev),
                   scores=torch.empty((B, J), dtype=torch.float32, device=dev)
                   if want_scores else None)
    workspace = _workspace(workspace, draft_verify_workspace_bytes(B, K, L, J, V), dev)
    itk = None
    if inv_temp_per_draft is not None:
        itk = (C.c_float * K)(*[float(x) for x in inv_temp_per_draft])
    _check(L_.gls_draft_verify(
        C.byref(drows), C.byref(trows), B, K, L, V, float(inv_temp),
        C.cast(itk, C.c_void_p) if itk is not None else None,
        float(inv_temp if inv_temp_target is None else inv_temp_target), C.byref(nz), int(flags),
        _ptr(out_draft_tokens), _ptr(out_draft_scores), _ptr(out["tokens"]), _ptr(out["tau"]),
        _ptr(out["accept"]), _ptr(out.get("scores")), workspace.data_ptr(), workspace.numel(),
        _ptr(status), _stream()))
    return out_draft_tokens, out_draft_scores, out


def compress_select(enc_logw, dec_logw=None, bins=None, K=None, seed=0, seq_base=0, seq_ids=None,
                    pos_base=0, spec=4, rounds=10, noise_flags=0, want_scores=True, workspace=None,
                    status=None, out=None):
    """enc_logw [B,N], dec_logw [B,K,N] | None, bins uint8 [N] | [B,N] | None.

    Returns dict(enc_index [B], message [B], dec_index [B,K], match [B], scores [B,1+K] | None)."""
    L = load()
    B, N = enc_logw.shape
    dev = enc_logw.device
    erows = _rows(enc_logw, 1)
    drows = None
    if dec_logw is not None:
        assert dec_logw.shape[0] == B and dec_logw.shape[2] == N
        K = dec_logw.shape[1]
        drows = _rows(dec_logw, 2)
    assert K is not None
    bsb = 0
    if bins is not None:
        if bins.dtype != torch.uint8 or not bins.is_contiguous():
            raise GlsError("bins must be contiguous uint8")
        bsb = 0 if bins.dim() == 1 else N
    nz = _noise(seed, seq_base, seq_ids, pos_base, spec, rounds, noise_flags)
    if out is None:
        out = dict(enc_index=torch.empty((B,), dtype=torch.int32, device=dev),
                   message=torch.empty((B,), dtype=torch.uint8, device=dev),
                   dec_index=torch.full((B, K), -1, dtype=torch.int32, device=dev),
                   match=torch.zeros((B,), dtype=torch.uint8, device=dev),
                   scores=torch.full((B, 1 + K), float("nan"), dtype=torch.float32, device=dev)
                   if want_scores else None)
    need = workspace_bytes(B, K, 1, N)
    workspace = _workspace(workspace, need, dev)
    _check(L.gls_compress_select(
        C.byref(erows), C.byref(drows) if drows is not None else None, _ptr(bins), bsb, B, K, N,
        C.byref(nz), _ptr(out["enc_index"]), _ptr(out["message"]), _ptr(out["dec_index"]),
        _ptr(out["match"]), _ptr(out.get("scores")), workspace.data_ptr(), workspace.numel(),
        _ptr(status), _stream()))
    return out


def compress_gaussian_workspace_bytes(B, K, N):
    return int(load().gls_compress_gaussian_workspace_bytes(int(B), int(K), int(N)))


def compress_gaussian(candidates, source, side_info, bins=None, s2_eta=0.5, s2_zeta=0.25,
                      s2_prior=1.0, seed=0, seq_base=0, seq_ids=None, pos_base=0, spec=4, rounds=10,
                      noise_flags=0, want_scores=True, workspace=None, status=None, out=None):
    """gls_compress_gaussian: candidates [N,D], source [B,D], side_info [B,K,D] (fp32, device).

    Returns compress_select's dict plus recon [B,K,D] and sqerr [B,K]."""
    L = load()
    N, D = candidates.shape
    B, K, _ = side_info.shape
    for x in (candidates, source, side_info):
        if not x.is_cuda or x.dtype != torch.float32 or not x.is_contiguous():
            raise GlsError("candidates, source and side_info must be contiguous float32 device tensors")
    assert tuple(source.shape) == (B, D) and tuple(side_info.shape) == (B, K, D)
    dev = candidates.device
    bsb = 0
    if bins is not None:
        if bins.dtype != torch.uint8 or not bins.is_contiguous():
            raise GlsError("bins must be contiguous uint8")
        bsb = 0 if bins.dim() == 1 else N
    nz = _noise(seed, seq_base, seq_ids, pos_base, spec, rounds, noise_flags)
    if out is None:
        out = dict(enc_index=torch.empty((B,), dtype=torch.int32, device=dev),
                   message=torch.empty((B,), dtype=torch.uint8, device=dev),
                   dec_index=torch.full((B, K), -1, dtype=torch.int32, device=dev),
                   match=torch.zeros((B,), dtype=torch.uint8, device=dev),
                   scores=torch.full((B, 1 + K), float("nan"), dtype=torch.float32, device=dev)
                   if want_scores else None,
                   recon=torch.empty((B, K, D), dtype=torch.float32, device=dev),
                   sqerr=torch.empty((B, K), dtype=torch.float32, device=dev))
    workspace = _workspace(workspace, compress_gaussian_workspace_bytes(B, K, N), dev)
    _check(L.gls_compress_gaussian(
        candidates.data_ptr(), source.data_ptr(), side_info.data_ptr(), _ptr(bins), bsb, B, K, N, D,
        float(s2_eta), float(s2_zeta), float(s2_prior), C.byref(nz), _ptr(out["enc_index"]),
        _ptr(out["message"]), _ptr(out["dec_index"]), _ptr(out["match"]), _ptr(out.get("scores")),
        _ptr(out.get("recon")), _ptr(out.get("sqerr")), workspace.data_ptr(), workspace.numel(),
        _ptr(status), _stream()))
    return out
