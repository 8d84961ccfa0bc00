"""ctypes binding: same names as the C ABI, argument marshalling only."""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
lib_path = os.path.join(_HERE, "libaser.so")

EXPORTED_SYMBOLS = (
    "aser_pack_w4", "aser_repacked_bytes", "aser_repack_w4", "aser_unrepack_w4",
    "aser_quant_act", "aser_quant_act_bits", "aser_quant_act_ex", "aser_quant_act_ws",
    "aser_quant_workspace_bytes", "aser_quant_act_ws_launches", "aser_forward_act_launches", "aser_linear_w4a8_lr_ld", "aser_forward_shared",
    "aser_linear_w4a8_lr_cat", "aser_forward_shared_cat_workspace_bytes", "aser_forward_shared_cat",
    "aser_forward_shared_workspace_bytes", "aser_construct", "aser_construct_workspace_bytes", "aser_linear_w4a8_lr", "aser_linear_w4a8", "aser_linear_w4a8_lr_simt", "aser_linear_w4a8_lr_static",
    "aser_workspace_bytes", "aser_workspace_init", "aser_check_status", "aser_forward",
    "aser_forward_host",
    "aser_last_error", "aser_version",
)

if not os.path.exists(lib_path):
    raise ImportError(
        f"{lib_path} is missing: build it with `python -m paper_2411_07762_b200.build` "
        "(there is no fallback path)")
lib = C.CDLL(lib_path)

_P, _I, _Z = C.c_void_p, C.c_int, C.c_size_t
lib.aser_pack_w4.argtypes = [_P, _P, _I, _I, _P, _P, _P]
lib.aser_repacked_bytes.argtypes = [_I, _I]
lib.aser_repacked_bytes.restype = _Z
lib.aser_repack_w4.argtypes = [_P, _I, _I, _P, _P]
lib.aser_unrepack_w4.argtypes = [_P, _I, _I, _P, _P]
lib.aser_quant_act.argtypes = [_P, _P, _P, _I, _I, _I, _P, _P, _P, _P]
lib.aser_quant_act_bits.argtypes = [_P, _P, _P, _I, _I, _I, _I, _P, _P, _P, _P]
lib.aser_quant_act_ex.argtypes = [_P, _P, _P, _I, _I, _I, _I, _I, _P, _P, _P, _P]
lib.aser_quant_workspace_bytes.argtypes = [_I, _I, _I]
lib.aser_quant_workspace_bytes.restype = _Z
lib.aser_forward_act_launches.argtypes = [_I, _I, _I]
lib.aser_forward_act_launches.restype = _I
lib.aser_quant_act_ws_launches.argtypes = [_I, _I]
lib.aser_quant_act_ws_launches.restype = _I
lib.aser_quant_act_ws.argtypes = [_P, _P, _P, _I, _I, _I, _I, _I, _P, _P, _P, _P, _Z, _P]
lib.aser_linear_w4a8_lr_ld.argtypes = [_P, _P, _P, _P, _P, _I, _P, _I, _I, _I, _I, _P, _P, _P, _Z, _P]
lib.aser_forward_shared_workspace_bytes.argtypes = [_I, _P, _P, _I, _I]
lib.aser_forward_shared_workspace_bytes.restype = _Z
lib.aser_forward_shared.argtypes = [_P, _P, _P, _I, _P, _P, _P, _P, _P, _I, _I, _P, _P, _P, _P, _P, _Z, _P]
lib.aser_linear_w4a8_lr_cat.argtypes = [_P, _P, _P, _P, _P, _P, _I, _P, _I, _I, _I, _P, _P, _Z, _P]
lib.aser_forward_shared_cat_workspace_bytes.argtypes = [_I, _P, _I, _I, _I]
lib.aser_forward_shared_cat_workspace_bytes.restype = _Z
lib.aser_forward_shared_cat.argtypes = [_P, _P, _P, _I, _P, _P, _P, _P, _I, _I, _I, _P, _P, _P, _P, _P, _Z, _P]
lib.aser_linear_w4a8_lr.argtypes = [_P, _P, _P, _P, _P, _P, _I, _I, _I, _I, _P, _P, _P, _Z, _P]
lib.aser_linear_w4a8.argtypes = [_P, _P, _P, _P, _I, _I, _I, _P, _P, _P, _Z, _P]
lib.aser_linear_w4a8_lr_simt.argtypes = [_P, _P, _P, _P, _P, _P, _I, _I, _I, _I, _P, _P, _P]
lib.aser_linear_w4a8_lr_static.argtypes = [_P, _P, _P, _P, _P, _P, _I, _I, _I, _I, _P, _P, _P]
lib.aser_workspace_bytes.argtypes = [_I, _I, _I, _I]
lib.aser_workspace_bytes.restype = _Z
lib.aser_workspace_init.argtypes = [_P, _Z, _P]
lib.aser_check_status.argtypes = [_P, _P]
lib.aser_forward.argtypes = [_P, _P, _P, _P, _P, _P, _I, _I, _I, _I, _P, _P, _P, _P, _P, _Z, _P]
lib.aser_forward_host.argtypes = [_P, _P, _P, _P, _P, _P, _P, _P, _P, _P, _P, _P,
                                  _I, _I, _I, _I, _P, _Z, _P]
lib.aser_construct_workspace_bytes.argtypes = [_I, _I, _I, _I, _I]
lib.aser_construct_workspace_bytes.restype = _Z
lib.aser_construct.argtypes = [_P, _P, _P, _I, _I, _I, _I, C.c_double, _I, _P, _P, _P, _P, _P, _P, _P, _I, _P, _Z, _P]
lib.aser_last_error.restype = C.c_char_p
lib.aser_version.restype = _I


class AserError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where} failed with code {code}: {last_error()}")


def last_error() -> str:
    return lib.aser_last_error().decode()


def version() -> int:
    return lib.aser_version()


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _chk(rc: int, where: str):
    if rc != 0:
        raise AserError(rc, where)


def _dev(t: torch.Tensor, dtype, name: str):
    if not t.is_cuda or t.dtype != dtype or not t.is_contiguous():
        raise TypeError(f"{name}: need a contiguous CUDA tensor of {dtype}")
    return t


def pack_w4(W: torch.Tensor, s: torch.Tensor | None):
    """W fp16 [N,K], s fp32 [K] or None -> (Wq uint8 [N,K/2] canonical, w_scale fp32 [N])."""
    _dev(W, torch.float16, "W")
    N, K = W.shape
    Wq = torch.empty((N, K // 2), dtype=torch.uint8, device=W.device)
    w_scale = torch.empty((N,), dtype=torch.float32, device=W.device)
    _chk(lib.aser_pack_w4(_ptr(W), _ptr(s), N, K, _ptr(Wq), _ptr(w_scale), _stream()), "aser_pack_w4")
    return Wq, w_scale


def repacked_bytes(N: int, K: int) -> int:
    return int(lib.aser_repacked_bytes(N, K))


def repack_w4(Wq: torch.Tensor) -> torch.Tensor:
    _dev(Wq, torch.uint8, "Wq")
    N, K = Wq.shape[0], Wq.shape[1] * 2
    Wk = torch.empty((repacked_bytes(N, K),), dtype=torch.uint8, device=Wq.device)
    _chk(lib.aser_repack_w4(_ptr(Wq), N, K, _ptr(Wk), _stream()), "aser_repack_w4")
    return Wk


def unrepack_w4(Wk: torch.Tensor, N: int, K: int) -> torch.Tensor:
    _dev(Wk, torch.uint8, "Wk")
    Wq = torch.empty((N, K // 2), dtype=torch.uint8, device=Wk.device)
    _chk(lib.aser_unrepack_w4(_ptr(Wk), N, K, _ptr(Wq), _stream()), "aser_unrepack_w4")
    return Wq


def quant_act(X: torch.Tensor, s: torch.Tensor | None, L_A: torch.Tensor | None,
              out=None, act_bits: int = 8, t_pair: bool = False):
    """X fp16 [M,K] -> (Xq int8 [M,K], a_scale fp32 [M], T bf16 [M,r]).  act_bits != 8 goes
    through aser_quant_act_bits (codes of that width in the int8 container); t_pair through
    aser_quant_act_ex (T [M,2r]: a bf16 value and its bf16 remainder per entry)."""
    _dev(X, torch.float16, "X")
    M, K = X.shape
    r = 0 if L_A is None else L_A.shape[0]
    if out is None:
        Xq = torch.empty((M, K), dtype=torch.int8, device=X.device)
        a_scale = torch.empty((M,), dtype=torch.float32, device=X.device)
        T = torch.empty((M, 2 * r if t_pair else r), dtype=torch.bfloat16, device=X.device)
    else:
        Xq, a_scale, T = out
    if t_pair:
        _chk(lib.aser_quant_act_ex(_ptr(X), _ptr(s), _ptr(L_A) if r else None, M, K, r, act_bits, 1,
                                   _ptr(Xq), _ptr(a_scale), _ptr(T) if r else None, _stream()),
             "aser_quant_act_ex")
        return Xq, a_scale, T
    if act_bits != 8:
        _chk(lib.aser_quant_act_bits(_ptr(X), _ptr(s), _ptr(L_A) if r else None, M, K, r, act_bits,
                                     _ptr(Xq), _ptr(a_scale), _ptr(T) if r else None, _stream()),
             "aser_quant_act_bits")
        return Xq, a_scale, T
    _chk(lib.aser_quant_act(_ptr(X), _ptr(s), _ptr(L_A) if r else None, M, K, r, _ptr(Xq),
                            _ptr(a_scale), _ptr(T) if r else None, _stream()), "aser_quant_act")
    return Xq, a_scale, T


def forward_act_launches(M: int, K: int, r: int) -> int:
    return int(lib.aser_forward_act_launches(M, K, r))


def quant_act_ws_launches(M: int, K: int) -> int:
    return int(lib.aser_quant_act_ws_launches(M, K))


def quant_workspace_bytes(M: int, K: int, r: int) -> int:
    return int(lib.aser_quant_workspace_bytes(M, K, r))


def quant_act_ws(X: torch.Tensor, s, L_A, ws: torch.Tensor | None = None, out=None,
                 act_bits: int = 8, t_pair: bool = False):
    """aser_quant_act_ws: quant_act with scratch memory (allocated here with torch when `ws` is
    None); L_A may be the stacked down projections of several layers, up to 512 rows."""
    _dev(X, torch.float16, "X")
    M, K = X.shape
    r = 0 if L_A is None else L_A.shape[0]
    if ws is None:
        ws = torch.empty((max(1024, quant_workspace_bytes(M, K, r)),), dtype=torch.uint8, device=X.device)
    if out is None:
        Xq = torch.empty((M, K), dtype=torch.int8, device=X.device)
        a_scale = torch.empty((M,), dtype=torch.float32, device=X.device)
        T = torch.empty((M, 2 * r if t_pair else r), dtype=torch.bfloat16, device=X.device)
    else:
        Xq, a_scale, T = out
    _chk(lib.aser_quant_act_ws(_ptr(X), _ptr(s), _ptr(L_A) if r else None, M, K, r, act_bits,
                               1 if t_pair else 0, _ptr(Xq), _ptr(a_scale), _ptr(T) if r else None,
                               _ptr(ws), ws.numel(), _stream()), "aser_quant_act_ws")
    return Xq, a_scale, T


def workspace_bytes(M: int, N: int, K: int, r: int) -> int:
    return int(lib.aser_workspace_bytes(M, N, K, r))


def new_workspace(M: int, N: int, K: int, r: int, device="cuda") -> torch.Tensor:
    """Allocate (with torch) and zero a workspace for the given problem size."""
    nbytes = max(256, workspace_bytes(M, N, K, r))
    ws = torch.empty((nbytes,), dtype=torch.uint8, device=device)
    _chk(lib.aser_workspace_init(_ptr(ws), nbytes, _stream()), "aser_workspace_init")
    return ws


def check_status(ws: torch.Tensor) -> None:
    _chk(lib.aser_check_status(_ptr(ws), _stream()), "aser_check_status")


def linear_w4a8_lr(Xq, a_scale, Wk, w_scale, T, L_B, N: int, ws: torch.Tensor,
                   Y=None, acc_debug=None):
    M, K = Xq.shape
    r = 0 if L_B is None else L_B.shape[1]
    if Y is None:
        Y = torch.empty((M, N), dtype=torch.float16, device=Xq.device)
    _chk(lib.aser_linear_w4a8_lr(_ptr(Xq), _ptr(a_scale), _ptr(Wk), _ptr(w_scale),
                                 _ptr(T) if r else None, _ptr(L_B) if r else None, M, N, K, r,
                                 _ptr(Y), _ptr(acc_debug), _ptr(ws), ws.numel(), _stream()),
         "aser_linear_w4a8_lr")
    return Y


def linear_w4a8_lr_ld(Xq, a_scale, Wk, w_scale, T_wide, col0: int, L_B, N: int, ws: torch.Tensor,
                      Y=None, acc_debug=None):
    """aser_linear_w4a8_lr_ld: the layer's T is columns [col0, col0 + r) of T_wide [M, R]."""
    M, K = Xq.shape
    r = L_B.shape[1]
    if Y is None:
        Y = torch.empty((M, N), dtype=torch.float16, device=Xq.device)
    t_ptr = C.c_void_p(T_wide.data_ptr() + 2 * col0)
    _chk(lib.aser_linear_w4a8_lr_ld(_ptr(Xq), _ptr(a_scale), _ptr(Wk), _ptr(w_scale), t_ptr,
                                    T_wide.shape[1], _ptr(L_B), M, N, K, r, _ptr(Y), _ptr(acc_debug),
                                    _ptr(ws), ws.numel(), _stream()), "aser_linear_w4a8_lr_ld")
    return Y


def linear_w4a8(Xq, a_scale, Wk, w_scale, N: int, ws: torch.Tensor, Y=None, acc_debug=None):
    M, K = Xq.shape
    if Y is None:
        Y = torch.empty((M, N), dtype=torch.float16, device=Xq.device)
    _chk(lib.aser_linear_w4a8(_ptr(Xq), _ptr(a_scale), _ptr(Wk), _ptr(w_scale), M, N, K, _ptr(Y),
                              _ptr(acc_debug), _ptr(ws), ws.numel(), _stream()), "aser_linear_w4a8")
    return Y


def linear_w4a8_lr_simt(Xq, a_scale, Wq, w_scale, T, L_B, Y=None, acc_debug=None):
    M, K = Xq.shape
    N = Wq.shape[0]
    r = 0 if L_B is None else L_B.shape[1]
    if Y is None:
        Y = torch.empty((M, N), dtype=torch.float16, device=Xq.device)
    _chk(lib.aser_linear_w4a8_lr_simt(_ptr(Xq), _ptr(a_scale), _ptr(Wq), _ptr(w_scale),
                                      _ptr(T) if r else None, _ptr(L_B) if r else None, M, N, K, r,
                                      _ptr(Y), _ptr(acc_debug), _stream()),
         "aser_linear_w4a8_lr_simt")
    return Y


def linear_w4a8_lr_static(Xq, a_scale, Wk, w_scale, T, L_B, N: int, Y=None, acc_debug=None):
    """aser_linear_w4a8_lr_static: same result as linear_w4a8_lr, no workspace argument (the
    library's built-in scratch array is used; at most 32 tokens per call)."""
    M, K = Xq.shape
    r = 0 if L_B is None else L_B.shape[1]
    if Y is None:
        Y = torch.empty((M, N), dtype=torch.float16, device=Xq.device)
    _chk(lib.aser_linear_w4a8_lr_static(_ptr(Xq), _ptr(a_scale), _ptr(Wk), _ptr(w_scale),
                                        _ptr(T) if r else None, _ptr(L_B) if r else None, M, N, K,
                                        r, _ptr(Y), _ptr(acc_debug), _stream()),
         "aser_linear_w4a8_lr_static")
    return Y


def construct(W: torch.Tensor, s, X_cal: torch.Tensor, r: int, damping: float = 0.01, iterations: int = 0,
              want_S: bool = False, split_idx: torch.Tensor | None = None):
    """aser_construct: int4 weights and rank-r factors of one layer built on the device from W
    fp16 [N,K], s fp32 [K] and calibration tokens fp16 [n_cal,K].  Returns a dict with Wq, w_scale,
    L_A fp16 [r,K], L_B fp16 [N,r], sigma fp64 [r] and (want_S) the whitening factor S fp64 [K,K]."""
    _dev(W, torch.float16, "W")
    _dev(X_cal, torch.float16, "X_cal")
    N, K = W.shape
    n_cal = X_cal.shape[0]
    dev = W.device
    Wq = torch.empty((N, K // 2), dtype=torch.uint8, device=dev)
    w_scale = torch.empty((N,), dtype=torch.float32, device=dev)
    L_A = torch.empty((max(r, 1), K), dtype=torch.float16, device=dev)
    L_B = torch.empty((N, max(r, 1)), dtype=torch.float16, device=dev)
    sigma = torch.empty((max(r, 1),), dtype=torch.float64, device=dev)
    S = torch.empty((K, K), dtype=torch.float64, device=dev) if want_S else None
    n_split = 0 if split_idx is None else int(split_idx.numel())
    if n_split:
        _dev(split_idx, torch.int32, "split_idx")
    nbytes = int(lib.aser_construct_workspace_bytes(N, K, n_cal, r, n_split))
    ws = torch.empty((max(nbytes, 256),), dtype=torch.uint8, device=dev)
    _chk(lib.aser_construct(_ptr(W), _ptr(s), _ptr(X_cal), N, K, n_cal, r, float(damping), int(iterations),
                            _ptr(Wq), _ptr(w_scale), _ptr(L_A), _ptr(L_B), _ptr(sigma), _ptr(S),
                            _ptr(split_idx) if n_split else None, n_split, _ptr(ws),
                            ws.numel(), _stream()), "aser_construct")
    return dict(Wq=Wq, w_scale=w_scale, L_A=L_A[:r], L_B=L_B[:, :r].contiguous(), sigma=sigma[:r], S=S)


def pair_up_projection(L_B: torch.Tensor) -> torch.Tensor:
    """[L_B | L_B]: the up projection a linear kernel needs beside a T stored as bf16 pairs."""
    return torch.cat([L_B, L_B], dim=1).contiguous()


def pad_rank(L_A: torch.Tensor, L_B: torch.Tensor, multiple: int = 16):
    """Factors of a rank that is not a multiple of 16 (a per-layer rank chosen by the paper's
    singular-value threshold, Sec. 4.1) -> the same factors with zero rows appended to L_A
    [r,K] and zero columns to L_B [N,r], which adds exact zeros to T L_B^T.  The kernels take
    ranks in steps of 16 up to 256."""
    r = L_A.shape[0]
    if L_B.shape[1] != r:
        raise ValueError("L_A has %d rows but L_B has %d columns" % (r, L_B.shape[1]))
    rp = (r + multiple - 1) // multiple * multiple
    if rp == r:
        return L_A.contiguous(), L_B.contiguous()
    A = torch.zeros((rp, L_A.shape[1]), dtype=L_A.dtype, device=L_A.device)
    B = torch.zeros((L_B.shape[0], rp), dtype=L_B.dtype, device=L_B.device)
    A[:r] = L_A
    B[:, :r] = L_B
    return A, B


class AserLinear:
    """Device-resident operands of one ASER-quantized linear layer plus preallocated
    intermediates for up to `max_tokens` tokens.  __call__ runs aser_quant_act followed by
    aser_linear_w4a8_lr on the current stream."""

    def __init__(self, W: torch.Tensor, s: torch.Tensor | None, L_A: torch.Tensor | None,
                 L_B: torch.Tensor | None, max_tokens: int):
        self.N, self.K = W.shape
        self.r = 0 if L_A is None else L_A.shape[0]
        self.s, self.L_A, self.L_B = s, L_A, L_B
        self.Wq, self.w_scale = pack_w4(W, s)
        self.Wk = repack_w4(self.Wq)
        dev = W.device
        self.max_tokens = max_tokens
        self.Xq = torch.empty((max_tokens, self.K), dtype=torch.int8, device=dev)
        self.a_scale = torch.empty((max_tokens,), dtype=torch.float32, device=dev)
        self.T = torch.empty((max_tokens, max(self.r, 1)), dtype=torch.bfloat16, device=dev)
        self.Y = torch.empty((max_tokens, self.N), dtype=torch.float16, device=dev)
        self.X_dev = torch.empty((max_tokens, self.K), dtype=torch.float16, device=dev)
        self.ws = new_workspace(max_tokens, self.N, self.K, self.r, dev)

    def quant(self, X: torch.Tensor):
        """The activation step alone, with the kernels aser_forward runs at this shape."""
        M = X.shape[0]
        r = self.r
        if forward_act_launches(M, self.K, r) == 1:
            _chk(lib.aser_quant_act(_ptr(X), _ptr(self.s), _ptr(self.L_A) if r else None, M, self.K, r,
                                    _ptr(self.Xq), _ptr(self.a_scale), _ptr(self.T) if r else None,
                                    _stream()), "aser_quant_act")
            return
        _chk(lib.aser_quant_act_ws(_ptr(X), _ptr(self.s), _ptr(self.L_A) if r else None, M, self.K, r,
                                   8, 0, _ptr(self.Xq), _ptr(self.a_scale), _ptr(self.T) if r else None,
                                   _ptr(self.ws), self.ws.numel(), _stream()), "aser_quant_act_ws")

    def linear(self, M: int, lowrank: bool = True, acc_debug=None):
        r = self.r if lowrank else 0
        if r:
            _chk(lib.aser_linear_w4a8_lr(_ptr(self.Xq), _ptr(self.a_scale), _ptr(self.Wk),
                                         _ptr(self.w_scale), _ptr(self.T), _ptr(self.L_B), M, self.N,
                                         self.K, r, _ptr(self.Y), _ptr(acc_debug), _ptr(self.ws),
                                         self.ws.numel(), _stream()), "aser_linear_w4a8_lr")
        else:
            _chk(lib.aser_linear_w4a8(_ptr(self.Xq), _ptr(self.a_scale), _ptr(self.Wk),
                                      _ptr(self.w_scale), M, self.N, self.K, _ptr(self.Y),
                                      _ptr(acc_debug), _ptr(self.ws), self.ws.numel(), _stream()),
                 "aser_linear_w4a8")

    def __call__(self, X: torch.Tensor, lowrank: bool = True) -> torch.Tensor:
        """One forward pass through aser_forward (quantization and linear kernel overlapped)."""
        M = X.shape[0]
        assert M <= self.max_tokens
        r = self.r if lowrank else 0       # the plain W4A8 control: the same entry point at rank 0
        _chk(lib.aser_forward(_ptr(X), _ptr(self.s), _ptr(self.L_A) if r else None, _ptr(self.Wk),
                              _ptr(self.w_scale), _ptr(self.L_B) if r else None, M, self.N, self.K, r,
                              _ptr(self.Xq), _ptr(self.a_scale), _ptr(self.T) if r else None,
                              _ptr(self.Y), _ptr(self.ws), self.ws.numel(), _stream()), "aser_forward")
        return self.Y[:M]

    def forward_host(self, X_host: torch.Tensor, Y_host: torch.Tensor):
        """Host fp16 X [M,K] (pinned) -> host fp16 Y [M,N] through aser_forward_host."""
        forward_host(self, X_host, Y_host)


class AserSharedInput:
    """Layers that read the same activation and share the smoothing vector (query/key/value, or
    gate/up): one activation pass for all of them through aser_forward_shared.  Built from
    AserLinear objects; their packed weights and factors are used in place."""

    def __init__(self, layers, max_tokens: int):
        self.layers = list(layers)
        first = self.layers[0]
        self.K, self.s = first.K, first.s
        for L in self.layers:
            if L.K != self.K or (L.s is not first.s and not torch.equal(L.s, first.s)):
                raise ValueError("layers of a shared-input group need the same K and smoothing vector")
        dev = first.Wk.device
        self.n = len(self.layers)
        self.r = [L.r for L in self.layers]
        self.N = [L.N for L in self.layers]
        self.r_total = sum(self.r)
        self.L_A = torch.cat([L.L_A for L in self.layers if L.r], dim=0).contiguous() if self.r_total else None
        self.max_tokens = max_tokens
        self.Xq = torch.empty((max_tokens, self.K), dtype=torch.int8, device=dev)
        self.a_scale = torch.empty((max_tokens,), dtype=torch.float32, device=dev)
        self.T = torch.empty((max_tokens, max(self.r_total, 1)), dtype=torch.bfloat16, device=dev)
        self.Y = [torch.empty((max_tokens, n), dtype=torch.float16, device=dev) for n in self.N]
        arr_i = C.c_int * self.n
        arr_p = C.c_void_p * self.n
        self._N, self._r = arr_i(*self.N), arr_i(*self.r)
        self._Wk = arr_p(*[L.Wk.data_ptr() for L in self.layers])
        self._ws = arr_p(*[L.w_scale.data_ptr() for L in self.layers])
        self._LB = arr_p(*[(L.L_B.data_ptr() if L.r else None) for L in self.layers])
        self._Y = arr_p(*[y.data_ptr() for y in self.Y])
        nbytes = int(lib.aser_forward_shared_workspace_bytes(self.n, self._N, self._r, max_tokens, self.K))
        if nbytes == 0:
            raise ValueError("unsupported shapes for a shared-input group")
        self.ws = torch.empty((nbytes,), dtype=torch.uint8, device=dev)
        _chk(lib.aser_workspace_init(_ptr(self.ws), nbytes, _stream()), "aser_workspace_init")

    def quant(self, X: torch.Tensor):
        """The activation pass of the group alone (aser_quant_act_ws with the stacked L_A)."""
        M = X.shape[0]
        if forward_act_launches(M, self.K, self.r_total) == 1 and self.r_total <= 256:
            _chk(lib.aser_quant_act(_ptr(X), _ptr(self.s), _ptr(self.L_A), M, self.K, self.r_total,
                                    _ptr(self.Xq), _ptr(self.a_scale), _ptr(self.T) if self.r_total else None,
                                    _stream()), "aser_quant_act")
            return
        _chk(lib.aser_quant_act_ws(_ptr(X), _ptr(self.s), _ptr(self.L_A), M, self.K, self.r_total, 8, 0,
                                   _ptr(self.Xq), _ptr(self.a_scale), _ptr(self.T) if self.r_total else None,
                                   _ptr(self.ws), self.ws.numel(), _stream()), "aser_quant_act_ws")

    def __call__(self, X: torch.Tensor):
        """Returns the layers' outputs [M, N_l] (views of preallocated buffers)."""
        M = X.shape[0]
        assert M <= self.max_tokens
        T = self.T if M == self.max_tokens else self.T[:M]
        _chk(lib.aser_forward_shared(_ptr(X), _ptr(self.s), _ptr(self.L_A), self.n, self._Wk, self._ws,
                                     self._LB, self._N, self._r, M, self.K, _ptr(self.Xq),
                                     _ptr(self.a_scale), _ptr(self.T) if self.r_total else None, self._Y,
                                     _ptr(self.ws), self.ws.numel(), _stream()), "aser_forward_shared")
        return [y[:M] for y in self.Y]



class AserSharedInputCat(AserSharedInput):
    """A shared-input group stored as one fused projection: the layers' packed weights, scales and
    up projections are concatenated along N (copies are made here) and the outputs are column
    ranges of one [M, sum N] buffer, so that a single linear launch serves the group
    (aser_forward_shared_cat).  Needs every N a multiple of 128 and one rank for all layers."""

    def __init__(self, layers, max_tokens: int):
        super().__init__(layers, max_tokens)
        if len(set(self.r)) != 1 or any(n % 128 for n in self.N) or self.n > 4:
            raise ValueError("a concatenated group needs one rank, N multiples of 128 and at most four layers")
        dev = self.layers[0].Wk.device
        self.r1 = self.r[0]
        self.N_total = sum(self.N)
        self.Wk_cat = torch.cat([L.Wk.reshape(-1) for L in self.layers]).contiguous()
        self.w_scale_cat = torch.cat([L.w_scale for L in self.layers]).contiguous()
        self.L_B_cat = torch.cat([L.L_B for L in self.layers], dim=0).contiguous() if self.r1 else None
        self.Y_cat = torch.empty((max_tokens, self.N_total), dtype=torch.float16, device=dev)
        nbytes = int(lib.aser_forward_shared_cat_workspace_bytes(self.n, self._N, self.r1, max_tokens, self.K))
        if nbytes == 0:
            raise ValueError("unsupported shapes for a concatenated shared-input group")
        if nbytes > self.ws.numel():
            self.ws = torch.empty((nbytes,), dtype=torch.uint8, device=dev)
            _chk(lib.aser_workspace_init(_ptr(self.ws), nbytes, _stream()), "aser_workspace_init")

    def _views(self, M: int):
        out, col = [], 0
        for n in self.N:
            out.append(self.Y_cat[:M, col:col + n])
            col += n
        return out

    def linear(self, M: int):
        """The linear step alone on the codes and T of the last activation pass."""
        _chk(lib.aser_linear_w4a8_lr_cat(_ptr(self.Xq), _ptr(self.a_scale), _ptr(self.Wk_cat),
                                         _ptr(self.w_scale_cat), _ptr(self.T) if self.r1 else None,
                                         _ptr(self.L_B_cat) if self.r1 else None, self.n, self._N, self.r1,
                                         M, self.K, _ptr(self.Y_cat), _ptr(self.ws), self.ws.numel(),
                                         _stream()), "aser_linear_w4a8_lr_cat")
        return self._views(M)

    def __call__(self, X: torch.Tensor):
        """Returns the layers' outputs as column ranges of the fused output [M, sum N]."""
        M = X.shape[0]
        assert M == self.max_tokens, "the fused output buffer is laid out for max_tokens rows"
        _chk(lib.aser_forward_shared_cat(_ptr(X), _ptr(self.s), _ptr(self.L_A), self.n, _ptr(self.Wk_cat),
                                         _ptr(self.w_scale_cat), _ptr(self.L_B_cat) if self.r1 else None,
                                         self._N, self.r1, M, self.K, _ptr(self.Xq), _ptr(self.a_scale),
                                         _ptr(self.T) if self.r_total else None, _ptr(self.Y_cat),
                                         _ptr(self.ws), self.ws.numel(), _stream()), "aser_forward_shared_cat")
        return self._views(M)


def forward_host(layer: AserLinear, X_host: torch.Tensor, Y_host: torch.Tensor):
    M = X_host.shape[0]
    r = layer.r
    _chk(lib.aser_forward_host(_ptr(X_host), _ptr(Y_host), _ptr(layer.X_dev), _ptr(layer.Xq),
                               _ptr(layer.a_scale), _ptr(layer.T), _ptr(layer.Y), _ptr(layer.s),
                               _ptr(layer.L_A) if r else None, _ptr(layer.Wk), _ptr(layer.w_scale),
                               _ptr(layer.L_B) if r else None, M, layer.N, layer.K, r,
                               _ptr(layer.ws), layer.ws.numel(), _stream()), "aser_forward_host")
