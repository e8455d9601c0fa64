"""ctypes binding of include/ceca.h.  Argument marshalling only."""
import ctypes
import os

import numpy as np

from . import build as _build

CECA_1P = 1
CECA_2P = 2
UNFUSED, FUSED_AUTO, FUSED_SMEM, FUSED_TMEM, FUSED_BLOCK = 0, 1, 2, 3, 4
WS_CONSENSUS_FUSED = 1
WS_CONSENSUS_UNFUSED = 2
WS_LOGREG_GRAD = 3
WS_STEP_HOST = 4

EXPORTS = ["ceca_schedule", "ceca_gossip_sgd_step", "ceca_consensus_rounds", "dsgd_logreg_grad",
           "ceca_workspace_bytes", "ceca_read_status", "ceca_gossip_sgd_step_host", "ceca_status_string",
           "dsgd_logreg_grad_static", "dsgd_logreg_grad_static_capacity", "dsgd_lsq_grad",
           "ceca_fused_wait_selftest", "ceca_gossip_sgd_step_bf16", "dsgd_grad_shard_dots", "dsgd_grad_shard_sum",
           "dsgd_grad_shard_apply"]


class Round(ctypes.Structure):
    """Mirror of ceca_round_t."""
    _fields_ = [("n", ctypes.c_int32), ("tau", ctypes.c_int32), ("r", ctypes.c_int32),
                ("delta", ctypes.c_int32), ("n_r", ctypes.c_int32), ("payload", ctypes.c_int32),
                ("a_num", ctypes.c_int32), ("a_den", ctypes.c_int32),
                ("b_num", ctypes.c_int32), ("b_den", ctypes.c_int32),
                ("a", ctypes.c_double), ("b", ctypes.c_double)]


class CecaError(RuntimeError):
    def __init__(self, status, where):
        self.status = int(status)
        super().__init__("%s: %s (status %d)" % (where, ceca_status_string(status), status))


_lib = None


def library_path():
    return _build.LIB


def library():
    """Loads libceca_b200.so (building it first when it is missing or older than its sources)."""
    global _lib
    if _lib is not None:
        return _lib
    path = _build.build() if (_build.is_stale() and os.environ.get("CECA_NO_BUILD") != "1") else _build.LIB
    lib = ctypes.CDLL(path)
    vp, i32, i64, f32 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_float
    lib.ceca_schedule.argtypes = [i32, i32, i64, ctypes.POINTER(Round), vp, vp]
    lib.ceca_schedule.restype = ctypes.c_int
    lib.ceca_gossip_sgd_step.argtypes = [vp, vp, vp, vp, vp, i32, i64, i64, f32, i32, i64, vp]
    lib.ceca_gossip_sgd_step.restype = ctypes.c_int
    lib.ceca_gossip_sgd_step_bf16.argtypes = [vp, vp, vp, vp, vp, i32, i64, i64, i32, f32, i32, i64, vp]
    lib.ceca_gossip_sgd_step_bf16.restype = ctypes.c_int
    lib.ceca_consensus_rounds.argtypes = [vp, vp, vp, vp, i32, i64, i64, i32, i64, i32, i32, vp,
                                          ctypes.c_size_t, vp]
    lib.ceca_consensus_rounds.restype = ctypes.c_int
    lib.dsgd_logreg_grad.argtypes = [vp, vp, vp, vp, i64, vp, i32, i32, i64, i64, i32, vp,
                                     ctypes.c_size_t, vp]
    lib.dsgd_logreg_grad.restype = ctypes.c_int
    lib.dsgd_lsq_grad.argtypes = [vp, vp, vp, vp, vp, i64, vp, i32, i32, i64, i64, i32, vp, ctypes.c_size_t, vp]
    lib.dsgd_lsq_grad.restype = ctypes.c_int
    lib.dsgd_grad_shard_dots.argtypes = [vp, vp, vp, i32, i32, i64, i64, i64, vp]
    lib.dsgd_grad_shard_dots.restype = ctypes.c_int
    lib.dsgd_grad_shard_sum.argtypes = [vp, vp, i64, i32, vp]
    lib.dsgd_grad_shard_sum.restype = ctypes.c_int
    lib.dsgd_grad_shard_apply.argtypes = [vp, vp, vp, vp, vp, i32, i32, i64, i64, i64, i32, vp]
    lib.dsgd_grad_shard_apply.restype = ctypes.c_int
    lib.dsgd_logreg_grad_static.argtypes = [vp, vp, vp, vp, i64, vp, i32, i32, i64, i64, i32, vp]
    lib.dsgd_logreg_grad_static.restype = ctypes.c_int
    lib.dsgd_logreg_grad_static_capacity.argtypes = []
    lib.dsgd_logreg_grad_static_capacity.restype = ctypes.c_size_t
    lib.ceca_workspace_bytes.argtypes = [ctypes.c_int, i32, i32, i64]
    lib.ceca_workspace_bytes.restype = ctypes.c_size_t
    lib.ceca_fused_wait_selftest.argtypes = [vp, vp, i32, i64, i64, i32, vp, ctypes.c_size_t, vp]
    lib.ceca_fused_wait_selftest.restype = ctypes.c_int
    lib.ceca_read_status.argtypes = [vp, ctypes.POINTER(i32), vp]
    lib.ceca_read_status.restype = ctypes.c_int
    lib.ceca_gossip_sgd_step_host.argtypes = [vp, vp, vp, i32, i64, i64, f32, i32, i64, vp, ctypes.c_size_t]
    lib.ceca_gossip_sgd_step_host.restype = ctypes.c_int
    lib.ceca_status_string.argtypes = [ctypes.c_int]
    lib.ceca_status_string.restype = ctypes.c_char_p
    _lib = lib
    return lib


def ceca_status_string(status):
    return library().ceca_status_string(int(status)).decode()


def _check(status, where):
    if status != 0:
        raise CecaError(status, where)


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream):
    if stream is None:
        import torch
        return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    return ctypes.c_void_p(getattr(stream, "cuda_stream", stream))


def _matrix(t, name, n=None, cuda=True):
    """(n, d, ld) of a 2-D fp32 tensor whose rows are contiguous."""
    import torch
    if t.dtype != torch.float32 or t.dim() != 2 or t.stride(1) != 1:
        raise ValueError("%s must be a 2-D float32 tensor with unit column stride" % name)
    if cuda != t.is_cuda:
        raise ValueError("%s must live in %s memory" % (name, "device" if cuda else "host"))
    if n is not None and t.shape[0] != n:
        raise ValueError("%s has the wrong number of rows" % name)
    return t.shape[0], t.shape[1], t.stride(0) if t.shape[0] > 1 else max(t.stride(0), t.shape[1])


def ceca_schedule(n, variant, k, peers=True):
    """(Round, recv_from, send_to); the peer arrays are int32 numpy arrays (None when peers=False)."""
    rd = Round()
    recv = np.empty(max(n, 0), dtype=np.int32) if peers else None
    send = np.empty(max(n, 0), dtype=np.int32) if peers else None
    st = library().ceca_schedule(n, variant, k, ctypes.byref(rd),
                                 recv.ctypes.data if peers else None, send.ctypes.data if peers else None)
    _check(st, "ceca_schedule")
    return rd, recv, send


def ceca_gossip_sgd_step(X, Y, G, gamma, variant, k, X_out=None, Y_out=None, stream=None, drop_y=False):
    """One DSGD-CECA iteration on device tensors.  Outputs default to in place.  Returns (X_out, Y_out).
    Y = Y_out = None asks for the X-only update (n a power of two); drop_y=True passes Y_out = NULL
    with Y given (legal in the last round of a cycle, where the new y is never used)."""
    n, d, ld = _matrix(X, "X")
    X_out = X if X_out is None else X_out
    if Y_out is None and Y is not None and not drop_y:
        Y_out = Y   # (Y and Y_out both None: the X-only update, legal for n a power of two)
    for t, name in ((Y, "Y"), (G, "G"), (X_out, "X_out"), (Y_out, "Y_out")):
        if t is not None and _matrix(t, name, n) != (n, d, ld):
            raise ValueError("%s must have the shape and row stride of X" % name)
    st = library().ceca_gossip_sgd_step(_ptr(X), _ptr(Y), _ptr(G), _ptr(X_out), _ptr(Y_out), n, d, ld,
                                        float(gamma), variant, k, _stream(stream))
    _check(st, "ceca_gossip_sgd_step")
    return X_out, Y_out


def _matrix_of(t, name, dtype, n=None):
    """(n, d, ld) of a 2-D device tensor of the given dtype whose rows are contiguous."""
    if t.dtype != dtype or t.dim() != 2 or t.stride(1) != 1 or not t.is_cuda:
        raise ValueError("%s must be a 2-D %s device tensor with unit column stride" % (name, dtype))
    if n is not None and t.shape[0] != n:
        raise ValueError("%s has the wrong number of rows" % name)
    return t.shape[0], t.shape[1], t.stride(0) if t.shape[0] > 1 else max(t.stride(0), t.shape[1])


def ceca_gossip_sgd_step_bf16(X, Y, G, gamma, variant, k, X_out=None, Y_out=None, stream=None):
    """One DSGD-CECA iteration with G stored as bfloat16 and X, Y either float32 or bfloat16 (all the same).
    Outputs default to in place.  Returns (X_out, Y_out)."""
    import torch
    xy = X.dtype
    if xy not in (torch.float32, torch.bfloat16):
        raise ValueError("X must be float32 or bfloat16")
    n, d, ld = _matrix_of(X, "X", xy)
    X_out = X if X_out is None else X_out
    Y_out = Y if Y_out is None else Y_out
    for t, name, dt in ((Y, "Y", xy), (G, "G", torch.bfloat16), (X_out, "X_out", xy), (Y_out, "Y_out", xy)):
        if t is not None and _matrix_of(t, name, dt, n) != (n, d, ld):
            raise ValueError("%s must have the shape and row stride (in elements) of X" % name)
    st = library().ceca_gossip_sgd_step_bf16(_ptr(X), _ptr(Y), _ptr(G), _ptr(X_out), _ptr(Y_out), n, d, ld,
                                             int(xy == torch.bfloat16), float(gamma), variant, k, _stream(stream))
    _check(st, "ceca_gossip_sgd_step_bf16")
    return X_out, Y_out


def ceca_consensus_rounds(X, Y, variant, k0, rounds, fused, X_out=None, Y_out=None, workspace=None,
                          want_y=True, stream=None):
    """`rounds` CECA rounds on device tensors.  Returns (X_out, Y_out); Y_out is None when want_y is false."""
    n, d, ld = _matrix(X, "X")
    X_out = X if X_out is None else X_out
    if want_y and Y_out is None:
        if Y is None:
            raise ValueError("Y_out is needed when Y is None and want_y is true")
        Y_out = Y
    for t, name in ((Y, "Y"), (X_out, "X_out"), (Y_out, "Y_out")):
        if t is not None and _matrix(t, name, n) != (n, d, ld):
            raise ValueError("%s must have the shape and row stride of X" % name)
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    st = library().ceca_consensus_rounds(_ptr(X), _ptr(Y), _ptr(X_out), _ptr(Y_out), n, d, ld, variant, k0,
                                         rounds, int(fused), _ptr(workspace), ws_bytes, _stream(stream))
    _check(st, "ceca_consensus_rounds")
    return X_out, Y_out


def ceca_fused_wait_selftest(X, X_out, fused, workspace, stream=None):
    """Runs the named fused consensus kernel with a landing barrier that cannot complete (test suites only)."""
    n, d, ld = _matrix(X, "X")
    if _matrix(X_out, "X_out", n) != (n, d, ld):
        raise ValueError("X_out must have the shape and row stride of X")
    ws_bytes = workspace.numel() * workspace.element_size()
    st = library().ceca_fused_wait_selftest(_ptr(X), _ptr(X_out), n, d, ld, int(fused), _ptr(workspace), ws_bytes,
                                            _stream(stream))
    _check(st, "ceca_fused_wait_selftest")


def dsgd_logreg_grad(A, labels, X, Y, k, variant, G, workspace, stream=None):
    """Per-agent logistic gradient at the model iteration k selects; writes G and returns it."""
    import torch
    if A.dtype != torch.float32 or A.dim() != 3 or not A.is_contiguous() or not A.is_cuda:
        raise ValueError("A must be a contiguous 3-D float32 device tensor")
    n, m, d = A.shape
    if labels.dtype != torch.float32 or tuple(labels.shape) != (n, m) or not labels.is_contiguous():
        raise ValueError("labels must be a contiguous float32 [n, m] tensor")
    _, dx, ld = _matrix(X, "X", n)
    if dx != d:
        raise ValueError("X must have d columns")
    for t, name in ((Y, "Y"), (G, "G")):
        if t is not None and _matrix(t, name, n) != (n, d, ld):
            raise ValueError("%s must have the shape and row stride of X" % name)
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    st = library().dsgd_logreg_grad(_ptr(A), _ptr(labels), _ptr(X), _ptr(Y), k, _ptr(G), n, m, d, ld, variant,
                                    _ptr(workspace), ws_bytes, _stream(stream))
    _check(st, "dsgd_logreg_grad")
    return G


def dsgd_lsq_grad(A, B, X, Y, k, variant, G, workspace, noise=None, stream=None):
    """Per-agent least-squares gradient A_i^T (A_i z_i - b_i) (+ noise) at the model iteration k selects."""
    import torch
    if A.dtype != torch.float32 or A.dim() != 3 or not A.is_contiguous() or not A.is_cuda:
        raise ValueError("A must be a contiguous 3-D float32 device tensor")
    n, m, d = A.shape
    if B.dtype != torch.float32 or tuple(B.shape) != (n, m) or not B.is_contiguous():
        raise ValueError("B must be a contiguous float32 [n, m] tensor")
    _, dx, ld = _matrix(X, "X", n)
    if dx != d:
        raise ValueError("X must have d columns")
    for t, name in ((Y, "Y"), (G, "G"), (noise, "noise")):
        if t is not None and _matrix(t, name, n) != (n, d, ld):
            raise ValueError("%s must have the shape and row stride of X" % name)
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    st = library().dsgd_lsq_grad(_ptr(A), _ptr(B), _ptr(X), _ptr(Y), _ptr(noise), k, _ptr(G), n, m, d, ld, variant,
                                 _ptr(workspace), ws_bytes, _stream(stream))
    _check(st, "dsgd_lsq_grad")
    return G


def shard_columns(d, shards, index, multiple=4):
    """[c0, c1): the columns of shard `index` when d columns are cut into `shards` contiguous blocks whose
    boundaries are multiples of `multiple` (so that every block keeps vector alignment); the last block
    takes the remainder.  Integers only."""
    if not (0 <= index < shards) or d < 1 or multiple < 1:
        raise ValueError("bad shard request")
    units = (d + multiple - 1) // multiple
    lo = (units * index // shards) * multiple
    hi = d if index == shards - 1 else (units * (index + 1) // shards) * multiple
    return min(lo, d), min(hi, d)


def _shard3(A, name):
    """(n, m, w, lda) of a 3-D float32 device tensor whose last dimension is contiguous and whose first two
    dimensions are laid out as n*m rows of one stride (a column slice of a dense n x m x d tensor is)."""
    import torch
    if A.dtype != torch.float32 or A.dim() != 3 or not A.is_cuda or A.stride(2) != 1:
        raise ValueError("%s must be a 3-D float32 device tensor with unit column stride" % name)
    n, m, w = A.shape
    lda = A.stride(1)
    if m > 1 and n > 1 and A.stride(0) != m * lda:
        raise ValueError("%s: the sample rows of all agents must be equally spaced" % name)
    return n, m, w, lda


def dsgd_grad_shard_dots(A_shard, Z_shard, dots, stream=None):
    """dots[i, s] = <A_shard[i, s, :], Z_shard[i, :]> for one column shard."""
    n, m, w, lda = _shard3(A_shard, "A_shard")
    _, wz, ldz = _matrix(Z_shard, "Z_shard", n)
    if wz != w or tuple(dots.shape) != (n, m) or not dots.is_contiguous():
        raise ValueError("Z_shard must be [n, w] and dots a contiguous [n, m] tensor")
    st = library().dsgd_grad_shard_dots(_ptr(A_shard), _ptr(Z_shard), _ptr(dots), n, m, w, lda, ldz, _stream(stream))
    _check(st, "dsgd_grad_shard_dots")
    return dots


def dsgd_grad_shard_sum(total, part, first, stream=None):
    """total = part (first) or total += part: the sum over shards that share a GPU, in the caller's order."""
    if total.shape != part.shape or not total.is_contiguous() or not part.is_contiguous():
        raise ValueError("total and part must be contiguous tensors of one shape")
    st = library().dsgd_grad_shard_sum(_ptr(total), _ptr(part), total.numel(), int(bool(first)), _stream(stream))
    _check(st, "dsgd_grad_shard_sum")
    return total


def dsgd_grad_shard_apply(A_shard, targets, dots, G_shard, loss=0, noise_shard=None, stream=None):
    """Turns the summed dots into coefficients in place and writes the shard's columns of the gradient."""
    n, m, w, lda = _shard3(A_shard, "A_shard")
    _, wg, ldg = _matrix(G_shard, "G_shard", n)
    if wg != w or tuple(dots.shape) != (n, m) or tuple(targets.shape) != (n, m) or not targets.is_contiguous():
        raise ValueError("G_shard must be [n, w], dots and targets contiguous [n, m] tensors")
    if noise_shard is not None and _matrix(noise_shard, "noise_shard", n) != (n, w, ldg):
        raise ValueError("noise_shard must have the shape and row stride of G_shard")
    st = library().dsgd_grad_shard_apply(_ptr(A_shard), _ptr(targets), _ptr(dots), _ptr(noise_shard), _ptr(G_shard),
                                         n, m, w, lda, ldg, int(loss), _stream(stream))
    _check(st, "dsgd_grad_shard_apply")
    return G_shard


def dsgd_logreg_grad_static(A, labels, X, Y, k, variant, G, stream=None):
    """dsgd_logreg_grad without a workspace argument, for callers that cannot allocate device memory
    (no allocator at hand, or none that may be called at that point): the scratch space is a fixed
    32 MiB buffer inside the library.  Larger problems raise CecaError (status 7).  Calls on one
    device share that buffer, so they must not overlap on the GPU."""
    import torch
    if A.dtype != torch.float32 or A.dim() != 3 or not A.is_contiguous() or not A.is_cuda:
        raise ValueError("A must be a contiguous 3-D float32 device tensor")
    n, m, d = A.shape
    if labels.dtype != torch.float32 or tuple(labels.shape) != (n, m) or not labels.is_contiguous():
        raise ValueError("labels must be a contiguous float32 [n, m] tensor")
    _, dx, ld = _matrix(X, "X", n)
    if dx != d:
        raise ValueError("X must have d columns")
    for t, name in ((Y, "Y"), (G, "G")):
        if t is not None and _matrix(t, name, n) != (n, d, ld):
            raise ValueError("%s must have the shape and row stride of X" % name)
    st = library().dsgd_logreg_grad_static(_ptr(A), _ptr(labels), _ptr(X), _ptr(Y), k, _ptr(G), n, m, d, ld,
                                           variant, _stream(stream))
    _check(st, "dsgd_logreg_grad_static")
    return G


def dsgd_logreg_grad_static_capacity():
    return int(library().dsgd_logreg_grad_static_capacity())


def ceca_workspace_bytes(kind, n, m, d):
    return int(library().ceca_workspace_bytes(kind, n, m, d))


def ceca_read_status(workspace, stream=None):
    out = ctypes.c_int32(-1)
    _check(library().ceca_read_status(_ptr(workspace), ctypes.byref(out), _stream(stream)), "ceca_read_status")
    return out.value


def ceca_gossip_sgd_step_host(X, Y, G, gamma, variant, k, workspace):
    """The iteration on HOST tensors (updated in place), streamed through a DEVICE workspace."""
    n, d, ld = _matrix(X, "X", cuda=False)
    for t, name in ((Y, "Y"), (G, "G")):
        if t is not None and _matrix(t, name, n, cuda=False) != (n, d, ld):
            raise ValueError("%s must have the shape and row stride of X" % name)
    if not workspace.is_cuda:
        raise ValueError("workspace must be device memory")
    ws_bytes = workspace.numel() * workspace.element_size()
    st = library().ceca_gossip_sgd_step_host(_ptr(X), _ptr(Y), _ptr(G), n, d, ld, float(gamma), variant, k,
                                             _ptr(workspace), ws_bytes)
    _check(st, "ceca_gossip_sgd_step_host")
    return X, Y
