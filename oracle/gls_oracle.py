"""ctypes front end of the CPU oracle (oracle/gls_oracle.c).

TEST INFRASTRUCTURE ONLY: nothing in the CUDA product path may import this module.  It compiles
the C file with gcc on first use (into oracle/libgls_oracle.so) and exposes numpy-in / numpy-out
functions that mirror the three library entry points:

  draft_sample           Algorithm 1 third step / Algorithm 2 draft loop
  target_sample_verify   Algorithm 2 verification (Appendix B variant by flag)
  compress_select        Sec. 5.1 encoder / decoder index selection

Inputs are host numpy arrays: fp32 logits as float32, bf16 logits as uint16 bit patterns.
"""
import ctypes as C
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gls_oracle.c")
_LIB = os.path.join(_HERE, "libgls_oracle.so")
_lock = threading.Lock()
_lib = None

F32, BF16, F64 = 0, 1, 2
NOISE_SHARED_ACROSS_K = 1
COMBINE_ALL = 1
NO_BONUS = 2


def build(force=False):
    """Compile the oracle with gcc (OpenMP, -O2, strict IEEE: no fast-math)."""
    if not force and os.path.exists(_LIB) and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC):
        return _LIB
    tmp = _LIB + ".tmp%d" % os.getpid()
    cmd = ["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared", "-ffp-contract=off",
           "-o", tmp, _SRC, "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, _LIB)
    return _LIB


class _Noise(C.Structure):
    _fields_ = [("seed", C.c_uint64), ("seq_base", C.c_uint32), ("seq_ids", C.c_void_p),
                ("pos_base", C.c_uint32), ("noise_spec", C.c_uint32), ("rounds", C.c_uint32),
                ("flags", C.c_uint32)]


def lib():
    global _lib
    with _lock:
        if _lib is None:
            build()
            L = C.CDLL(_LIB)
            L.glso_uniform_flat.restype = C.c_double
            L.glso_uniform_flat.argtypes = [C.c_uint64, C.c_int, C.c_int, C.c_uint32, C.c_uint32,
                                            C.c_uint32, C.c_uint32, C.c_int64]
            L.glso_exp_noise_row.restype = None
            L.glso_exp_noise_row.argtypes = [C.c_uint64, C.c_int, C.c_int, C.c_uint32, C.c_uint32,
                                             C.c_uint32, C.c_uint32, C.c_int64, C.c_void_p]
            L.glso_row_lse.restype = C.c_double
            L.glso_row_lse.argtypes = [C.c_void_p, C.c_int, C.c_int64, C.c_double]
            L.glso_philox4x32.restype = None
            L.glso_philox4x32.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_void_p]
            L.glso_draft_sample.restype = C.c_int
            L.glso_target_sample_verify.restype = C.c_int
            L.glso_compress_select.restype = C.c_int
            L.glso_set_threads.argtypes = [C.c_int]
            L.glso_max_threads.restype = C.c_int
            _lib = L
    return _lib


def set_threads(n):
    lib().glso_set_threads(int(n))


def max_threads():
    return int(lib().glso_max_threads())


def philox4x32(ctr, key, rounds=10):
    c = np.ascontiguousarray(ctr, dtype=np.uint32)
    k = np.ascontiguousarray(key, dtype=np.uint32)
    out = np.empty(4, dtype=np.uint32)
    lib().glso_philox4x32(c.ctypes.data, k.ctypes.data, int(rounds), out.ctypes.data)
    return out


def uniform(seed, seq, pos, k, i, spec=4, domain=0, rounds=10):
    return float(lib().glso_uniform_flat(int(seed), int(rounds), int(spec), int(domain), int(seq),
                                         int(pos), int(k), int(i)))


def exp_noise(seed, seq, pos, k, i, spec=4, domain=0, rounds=10):
    f = lib().glso_exp_noise_flat
    f.restype = C.c_double
    return float(f(C.c_uint64(int(seed)), C.c_int(int(rounds)), C.c_int(int(spec)), C.c_uint32(int(domain)),
                   C.c_uint32(int(seq)), C.c_uint32(int(pos)), C.c_uint32(int(k)), C.c_int64(int(i))))


def exp_noise_row(seed, seq, pos, k, V, spec=4, domain=0, rounds=10):
    """S_i = -ln U_i for i < V under one (sequence, position, draft) key, fp64."""
    out = np.empty(int(V), dtype=np.float64)
    lib().glso_exp_noise_row(int(seed), int(rounds), int(spec), int(domain), int(seq), int(pos),
                             int(k), int(V), out.ctypes.data)
    return out


def exp_noise_batch(seed, B, K, V, pos=0, seq_base=0, spec=4, domain=0, rounds=10):
    """S[b,k,i] for sequences seq_base..seq_base+B-1, drafts 0..K-1, one position, fp64."""
    out = np.empty((int(B), int(K), int(V)), dtype=np.float64)
    f = lib().glso_exp_noise_batch
    f.restype = None
    f(C.c_uint64(seed), C.c_int(rounds), C.c_int(spec), C.c_uint32(domain), C.c_uint32(seq_base),
      C.c_int(B), C.c_uint32(pos), C.c_int(K), C.c_int64(V), C.c_void_p(out.ctypes.data))
    return out


def row_lse(row, inv_temp=1.0):
    row, dt = _as_rows(row)
    return float(lib().glso_row_lse(row.ctypes.data, dt, row.shape[-1], float(inv_temp)))


def _as_rows(a):
    a = np.asarray(a)
    if a.dtype == np.float32:
        return a, F32
    if a.dtype == np.uint16:
        return a, BF16
    if a.dtype == np.float64:
        return a, F64
    raise TypeError("logits must be float32 or uint16 (bf16 bit patterns), got %s" % a.dtype)


def _strides_elems(a, ndim_lead):
    """Element strides of the leading dims of an array whose last dim is contiguous."""
    assert a.strides[-1] == a.itemsize, "token dimension must be contiguous"
    return [s // a.itemsize for s in a.strides[:ndim_lead]]


def _noise(seed, seq_base, seq_ids, pos_base, spec, rounds, flags):
    keep = None
    ptr = None
    if seq_ids is not None:
        keep = np.ascontiguousarray(seq_ids, dtype=np.uint32)
        ptr = keep.ctypes.data
    nz = _Noise(int(seed), int(seq_base), ptr, int(pos_base), int(spec), int(rounds), int(flags))
    return nz, keep


def draft_sample(logits, inv_temp=1.0, inv_temp_per_draft=None, seed=0, seq_base=0, seq_ids=None,
                 pos_base=0, spec=4, rounds=10, noise_flags=0):
    """logits [B,K,J,V] (strided views allowed) -> dict(tokens, scores, gaps), each [B,K,J]."""
    logits, dt = _as_rows(logits)
    B, K, J, V = logits.shape
    sb, sk, sj = _strides_elems(logits, 3)
    nz, keep = _noise(seed, seq_base, seq_ids, pos_base, spec, rounds, noise_flags)
    tokens = np.empty((B, K, J), dtype=np.int32)
    scores = np.empty((B, K, J), dtype=np.float64)
    gaps = np.empty((B, K, J), dtype=np.float64)
    itk = None
    if inv_temp_per_draft is not None:
        itk = np.ascontiguousarray(inv_temp_per_draft, dtype=np.float32)
        assert itk.shape == (K,)
    rc = lib().glso_draft_sample(
        C.c_void_p(logits.ctypes.data), C.c_int(dt), C.c_int64(sb), C.c_int64(sk), C.c_int64(sj),
        C.c_int(B), C.c_int(K), C.c_int(J), C.c_int64(V), C.c_float(inv_temp),
        C.c_void_p(itk.ctypes.data if itk is not None else None), C.byref(nz),
        C.c_void_p(tokens.ctypes.data), C.c_void_p(scores.ctypes.data),
        C.c_void_p(gaps.ctypes.data))
    if rc != 0:
        raise ValueError("oracle draft_sample: invalid arguments")
    return dict(tokens=tokens, scores=scores, gaps=gaps)


def target_sample_verify(logits, draft_tokens, inv_temp=1.0, flags=0, seed=0, seq_base=0,
                         seq_ids=None, pos_base=0, spec=4, rounds=10, noise_flags=0):
    """logits [B,K,J,V], draft_tokens [B,K,L] with J = L+1 (L with NO_BONUS).

    Returns dict(tokens [B,J], tau [B], accept [B,K,L], scores [B,J], gaps [B,J], row_lse [B,K,J]).
    """
    logits, dt = _as_rows(logits)
    B, K, J, V = logits.shape
    L = J if (flags & NO_BONUS) else J - 1
    sb, sk, sj = _strides_elems(logits, 3)
    dtok = np.ascontiguousarray(draft_tokens, dtype=np.int32).reshape(B, K, L)
    nz, keep = _noise(seed, seq_base, seq_ids, pos_base, spec, rounds, noise_flags)
    tokens = np.empty((B, J), dtype=np.int32)
    tau = np.empty((B,), dtype=np.int32)
    accept = np.zeros((B, K, max(L, 0)), dtype=np.uint8)
    scores = np.empty((B, J), dtype=np.float64)
    gaps = np.empty((B, J), dtype=np.float64)
    rlse = np.empty((B, K, J), dtype=np.float64)
    rc = lib().glso_target_sample_verify(
        C.c_void_p(logits.ctypes.data), C.c_int(dt), C.c_int64(sb), C.c_int64(sk), C.c_int64(sj),
        C.c_int(B), C.c_int(K), C.c_int(L), C.c_int64(V), C.c_float(inv_temp),
        C.c_void_p(dtok.ctypes.data if L > 0 else None), C.byref(nz), C.c_uint32(flags),
        C.c_void_p(tokens.ctypes.data), C.c_void_p(tau.ctypes.data),
        C.c_void_p(accept.ctypes.data if L > 0 else None), C.c_void_p(scores.ctypes.data),
        C.c_void_p(gaps.ctypes.data), C.c_void_p(rlse.ctypes.data))
    if rc != 0:
        raise ValueError("oracle target_sample_verify: invalid arguments")
    return dict(tokens=tokens, tau=tau, accept=accept, scores=scores, gaps=gaps, row_lse=rlse)


def compress_select(enc_logw, dec_logw=None, bins=None, seed=0, seq_base=0, seq_ids=None,
                    pos_base=0, spec=4, rounds=10, noise_flags=0, K=None):
    """enc_logw [B,N]; dec_logw [B,K,N] or None (then K must be given); bins None, [N] or [B,N].

    Returns dict(enc_index [B], message [B], dec_index [B,K], match [B], scores, gaps [B,1+K]).
    """
    enc, edt = _as_rows(enc_logw)
    B, N = enc.shape
    (esb,) = _strides_elems(enc, 1)
    if dec_logw is not None:
        dec, ddt = _as_rows(dec_logw)
        assert dec.shape[0] == B and dec.shape[2] == N
        K = dec.shape[1]
        dsb, dsk = _strides_elems(dec, 2)
        dptr = dec.ctypes.data
    else:
        assert K is not None
        ddt, dsb, dsk, dptr = F32, 0, 0, None
    bptr, bsb = None, 0
    if bins is not None:
        bins = np.ascontiguousarray(bins, dtype=np.uint8)
        bptr = bins.ctypes.data
        bsb = 0 if bins.ndim == 1 else N
        assert bins.shape[-1] == N
    nz, keep = _noise(seed, seq_base, seq_ids, pos_base, spec, rounds, noise_flags)
    enc_index = np.empty((B,), dtype=np.int32)
    message = np.empty((B,), dtype=np.uint8)
    dec_index = np.full((B, K), -1, dtype=np.int32)
    match = np.zeros((B,), dtype=np.uint8)
    scores = np.full((B, 1 + K), np.nan, dtype=np.float64)
    gaps = np.full((B, 1 + K), np.nan, dtype=np.float64)
    rc = lib().glso_compress_select(
        C.c_void_p(enc.ctypes.data), C.c_int(edt), C.c_int64(esb), C.c_void_p(dptr), C.c_int(ddt),
        C.c_int64(dsb), C.c_int64(dsk), C.c_void_p(bptr), C.c_int64(bsb), C.c_int(B), C.c_int(K),
        C.c_int64(N), C.byref(nz), C.c_void_p(enc_index.ctypes.data),
        C.c_void_p(message.ctypes.data), C.c_void_p(dec_index.ctypes.data),
        C.c_void_p(match.ctypes.data), C.c_void_p(scores.ctypes.data),
        C.c_void_p(gaps.ctypes.data))
    if rc != 0:
        raise ValueError("oracle compress_select: invalid arguments")
    return dict(enc_index=enc_index, message=message, dec_index=dec_index, match=match,
                scores=scores, gaps=gaps)


def compress_gaussian(u, a, t, bins=None, s2_eta=0.5, s2_zeta=0.25, s2_prior=1.0, seed=0,
                      seq_base=0, seq_ids=None, pos_base=0, spec=4, rounds=10, noise_flags=0,
                      want_logw=False):
    """Appendix C with the Gaussian model of Sec. 5.2 / Appendix D.3 (per dimension).

    u [N,D] candidates drawn from N(0, s2_prior I); a [B,D] sources; t [B,K,D] side information.
    Returns compress_select's dict plus recon [B,K,D], sqerr [B,K] (mean squared error per
    dimension of each decoder's reconstruction) and, on request, logw [B,1+K,N]."""
    u = np.ascontiguousarray(u, dtype=np.float32)
    a = np.ascontiguousarray(a, dtype=np.float32)
    t = np.ascontiguousarray(t, dtype=np.float32)
    N, D = u.shape
    B, K, _ = t.shape
    assert a.shape == (B, D) and t.shape == (B, K, D)
    bptr, bsb = None, 0
    if bins is not None:
        bins = np.ascontiguousarray(bins, dtype=np.uint8)
        bptr = bins.ctypes.data
        bsb = 0 if bins.ndim == 1 else N
        assert bins.shape[-1] == N
    nz, keep = _noise(seed, seq_base, seq_ids, pos_base, spec, rounds, noise_flags)
    out = dict(enc_index=np.empty((B,), np.int32), message=np.empty((B,), np.uint8),
               dec_index=np.full((B, K), -1, np.int32), match=np.zeros((B,), np.uint8),
               scores=np.full((B, 1 + K), np.nan), gaps=np.full((B, 1 + K), np.nan),
               recon=np.empty((B, K, D)), sqerr=np.empty((B, K)))
    logw = np.empty((B, 1 + K, N)) if want_logw else None
    f = lib().glso_compress_gaussian
    f.restype = C.c_int
    rc = f(C.c_void_p(u.ctypes.data), C.c_void_p(a.ctypes.data), C.c_void_p(t.ctypes.data),
           C.c_void_p(bptr), C.c_int64(bsb), C.c_int(B), C.c_int(K), C.c_int64(N), C.c_int(D),
           C.c_double(s2_eta), C.c_double(s2_zeta), C.c_double(s2_prior), C.byref(nz),
           C.c_void_p(out["enc_index"].ctypes.data), C.c_void_p(out["message"].ctypes.data),
           C.c_void_p(out["dec_index"].ctypes.data), C.c_void_p(out["match"].ctypes.data),
           C.c_void_p(out["scores"].ctypes.data), C.c_void_p(out["gaps"].ctypes.data),
           C.c_void_p(out["recon"].ctypes.data), C.c_void_p(out["sqerr"].ctypes.data),
           C.c_void_p(logw.ctypes.data if want_logw else None))
    if rc != 0:
        raise ValueError("oracle compress_gaussian: invalid arguments")
    if want_logw:
        out["logw"] = logw
    return out


def top_m_rows(logits, M):
    """Top-M truncation of dense rows (Sec. 4.4 / Appendix D.1: sampling from the M most likely
    tokens): per row keep the M largest finite logits, ties at the M-th value going to the lower
    token index, and set every other entry to -inf (a masked token).  NaN, +inf and -inf entries are
    never kept; a row with fewer than M finite entries keeps them all.

    logits: float array [..., V].  Returns (float32 array of the same shape, list of kept index
    arrays in ascending order, one per row in C order).  Plain sort per row: slow and obvious."""
    x = np.asarray(logits, dtype=np.float32)
    flat = x.reshape(-1, x.shape[-1])
    out = np.full_like(flat, -np.inf)
    kept = []
    for r in range(flat.shape[0]):
        cand = [(-float(v), i) for i, v in enumerate(flat[r]) if np.isfinite(v)]
        cand.sort()  # by logit descending, then index ascending
        k = np.array(sorted(i for _, i in cand[:M]), dtype=np.int64)
        out[r, k] = flat[r, k]
        kept.append(k)
    return out.reshape(x.shape), kept
