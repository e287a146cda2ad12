"""ctypes binding of liblq.so: the same entry points as include/lq.h, argument marshalling only.

Every step of the path runs inside the library's CUDA kernels; PyTorch appears only as the
owner of device buffers and streams.  If the shared library is missing the import of any entry
point raises - there is no CPU fallback.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "liblq.so")

LQ_OK = 0
BRANCH = {"none": 0, "w16a16": 1, "w8a8": 2, "w6a6": 3, "w4a8": 4, "mxfp8": 5, "mxfp6": 6, "mxfp4": 7,
          "mxint8": 8, "mxint4": 9}
MAIN_AUTO, MAIN_MXFP4, MAIN_MXINT4_A8 = 0, 2, 3
ACT_DEFAULT, ACT_MXFP6 = 0, 6
BRANCH_NAME = {v: k for k, v in BRANCH.items()}
OUT_F16, OUT_F32 = 0, 1
GROUP = 64


class LqConfig(C.Structure):
    _fields_ = [("K", C.c_int32), ("N", C.c_int32), ("rank", C.c_int32), ("group", C.c_int32),
                ("branch", C.c_int32), ("steps", C.c_int32), ("lr", C.c_float), ("beta1", C.c_float),
                ("beta2", C.c_float), ("eps", C.c_float), ("rot_steps", C.c_int32), ("rot_lr", C.c_float),
                ("seed", C.c_uint64), ("main_fmt", C.c_int32), ("act_fmt", C.c_int32)]


class LqError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        detail = f" [{lib().lq_last_cuda_error().decode()}]" if code == 4 else ""
        super().__init__(f"{where}: {lib().lq_status_string(code).decode()} (lq_status {code}){detail}")


_lib = None

_SIGNATURES = {
    "lq_config_default": [C.POINTER(LqConfig), C.c_int32, C.c_int32, C.c_int32, C.c_int32],
    "lq_calibrate": [C.POINTER(LqConfig), C.c_void_p, C.c_void_p, C.POINTER(C.c_void_p), C.c_void_p],
    "lq_layer_import": [C.POINTER(LqConfig), C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                        C.c_void_p, C.c_void_p, C.POINTER(C.c_void_p)],
    "lq_layer_export": [C.c_void_p] * 8,
    "lq_layer_info": [C.c_void_p, C.POINTER(LqConfig)],
    "lq_layer_to_device": [C.c_void_p, C.c_int],
    "lq_layer_free": [C.c_void_p],
    "lq_act_create": [C.c_void_p, C.c_int32, C.c_int, C.POINTER(C.c_void_p)],
    "lq_act_free": [C.c_void_p],
    "lq_quantize_act": [C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p],
    "lq_linear_forward": [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_void_p],
    "lq_linear_forward_host": [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_int, C.c_void_p],
    "lq_linear_forward_host_async": [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_int, C.c_void_p],
    "lq_linear_forward_static": [C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_int, C.c_void_p],
    "lq_act_export": [C.c_void_p] * 8,
    "lq_get_device_status": [C.c_int, C.POINTER(C.c_int32), C.POINTER(C.c_int32)],
    "lq_set_option": [C.c_char_p, C.c_int32],
    "lq_selftest_wait_timeout": [C.c_int, C.c_void_p],
}
EXPORTED = tuple(_SIGNATURES) + ("lq_status_string", "lq_last_cuda_error", "lq_version")


def lib() -> C.CDLL:
    """The loaded shared library (raises if it has not been built)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} not found: build it with `python -m paper_2604_18117_b200.build`")
        _lib = C.CDLL(LIB_PATH)
        for name, args in _SIGNATURES.items():
            fn = getattr(_lib, name)
            fn.argtypes = args
            fn.restype = C.c_int
        _lib.lq_status_string.argtypes = [C.c_int]
        _lib.lq_status_string.restype = C.c_char_p
        _lib.lq_last_cuda_error.argtypes = []
        _lib.lq_last_cuda_error.restype = C.c_char_p
        _lib.lq_version.argtypes = []
        _lib.lq_version.restype = C.c_int
    return _lib


def _check(code: int, where: str):
    if code != LQ_OK:
        raise LqError(code, where)


def _np_ptr(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def lq_config_default(K: int, N: int, rank: int, branch) -> LqConfig:
    cfg = LqConfig()
    b = BRANCH[branch] if isinstance(branch, str) else int(branch)
    _check(lib().lq_config_default(C.byref(cfg), K, N, rank, b), "lq_config_default")
    return cfg


def lq_calibrate(cfg: LqConfig, W16: np.ndarray, bias16: np.ndarray | None = None, want_trace: bool = False):
    """W16: fp16 [K, N] host array.  Returns (layer handle, trace or None)."""
    W16 = np.ascontiguousarray(W16, dtype=np.float16)
    assert W16.shape == (cfg.K, cfg.N)
    b = None if bias16 is None else np.ascontiguousarray(bias16, dtype=np.float16)
    trace = np.zeros(cfg.steps + 1, dtype=np.float64) if want_trace else None
    h = C.c_void_p()
    _check(lib().lq_calibrate(C.byref(cfg), _np_ptr(W16), _np_ptr(b), C.byref(h), _np_ptr(trace)), "lq_calibrate")
    return h, trace


def pack_nibbles(Wq: np.ndarray) -> np.ndarray:
    """int8 codes [K, N] -> bytes [K, N/2]: column 2j in the low nibble, 2j+1 in the high nibble."""
    u = Wq.astype(np.uint8) & 0xF
    return np.ascontiguousarray(u[:, 0::2] | (u[:, 1::2] << 4))


def unpack_nibbles(P: np.ndarray) -> np.ndarray:
    lo = (P & 0xF).astype(np.int8)
    hi = (P >> 4).astype(np.int8)
    lo = np.where(lo >= 8, lo - 16, lo).astype(np.int8)
    hi = np.where(hi >= 8, hi - 16, hi).astype(np.int8)
    out = np.empty((P.shape[0], P.shape[1] * 2), dtype=np.int8)
    out[:, 0::2], out[:, 1::2] = lo, hi
    return out


# ---- e4m3 / e2m1 byte formats (layout only: the bit patterns of the OCP element formats; no method arithmetic) ----
def _e4m3_table() -> np.ndarray:
    """Value of each of the 256 e4m3 bit patterns (bias 7, subnormals, no infinities; 0x7F / 0xFF are NaN)."""
    t = np.zeros(256, dtype=np.float32)
    for b in range(256):
        e, m = (b >> 3) & 0xF, b & 7
        v = m / 8.0 * 2.0 ** -6 if e == 0 else (1 + m / 8.0) * 2.0 ** (e - 7)
        t[b] = np.nan if (b & 0x7F) == 0x7F else (-v if b & 0x80 else v)
    return t


E4M3_VALUES = _e4m3_table()


def e4m3_decode(codes: np.ndarray) -> np.ndarray:
    """uint8 / int8 e4m3 bit patterns -> float32 values."""
    return E4M3_VALUES[np.asarray(codes).view(np.uint8)]


def e4m3_encode(values: np.ndarray) -> np.ndarray:
    """float values that are exactly representable in e4m3 -> their bit patterns (uint8); raises otherwise."""
    v = np.asarray(values, dtype=np.float32)
    pos = E4M3_VALUES[:0x7F]                                   # ascending non-negative values
    idx = np.searchsorted(pos, np.abs(v))
    idx = np.minimum(idx, 0x7E)
    if not np.array_equal(pos[idx], np.abs(v)):
        raise ValueError("value not representable in e4m3")
    return (idx.astype(np.uint8) | np.where(np.signbit(v), 0x80, 0).astype(np.uint8)).astype(np.uint8)


def pack_e2m1(values: np.ndarray) -> np.ndarray:
    """e2m1 element values [K, N] -> nibbles [K, N/2] (sign, two exponent bits, one mantissa bit), column 2j low."""
    grid = np.array([0, 0.5, 1, 1.5, 2, 3, 4, 6], dtype=np.float32)
    v = np.asarray(values, dtype=np.float32)
    idx = np.searchsorted(grid, np.abs(v))
    idx = np.minimum(idx, 7)
    if not np.array_equal(grid[idx], np.abs(v)):
        raise ValueError("value not representable in e2m1")
    nib = (idx | np.where(np.signbit(v) & (v != 0), 8, 0)).astype(np.uint8)
    return np.ascontiguousarray(nib[:, 0::2] | (nib[:, 1::2] << 4))


def lq_layer_import(cfg: LqConfig, Wq_packed, sw, L1=None, sL1=None, L2=None, sL2=None, bias=None):
    """All arguments are host numpy arrays in the layouts include/lq.h documents."""
    arrs = [np.ascontiguousarray(a) if a is not None else None for a in (Wq_packed, sw, L1, sL1, L2, sL2, bias)]
    h = C.c_void_p()
    _check(lib().lq_layer_import(C.byref(cfg), *[_np_ptr(a) for a in arrs], C.byref(h)), "lq_layer_import")
    return h


def lq_layer_info(layer) -> LqConfig:
    cfg = LqConfig()
    _check(lib().lq_layer_info(layer, C.byref(cfg)), "lq_layer_info")
    return cfg


def lq_layer_export(layer) -> dict:
    cfg = lq_layer_info(layer)
    K, N, r, G = cfg.K, cfg.N, cfg.rank, -(-cfg.K // cfg.group)
    out = {"Wq_packed": np.zeros((K, N // 2), np.uint8), "sw": np.zeros((G, N), np.float16),
           "bias": np.zeros(N, np.float16), "branch": BRANCH_NAME[cfg.branch], "rank": r, "K": K, "N": N}
    L1 = L2 = sL1 = sL2 = None
    if cfg.main_fmt == MAIN_MXFP4 and r > 0:
        L1, L2 = np.zeros((K, r), np.uint8), np.zeros((r, N), np.uint8)               # e4m3 bit patterns
        sL1, sL2 = np.zeros((G, r), np.float32), np.zeros((-(-r // 32), N), np.float32)
    elif cfg.main_fmt == MAIN_MXINT4_A8 and r > 0:
        L1, L2 = np.zeros((K, r), np.int8), np.zeros((r, N), np.int8)                 # integer codes
        sL1, sL2 = np.zeros((G, r), np.float32), np.zeros((-(-r // 32), N), np.float32)   # block scales 2^e
    elif r > 0 and cfg.branch == BRANCH["w16a16"]:
        L1, L2 = np.zeros((K, r), np.float16), np.zeros((r, N), np.float16)
    elif r > 0:
        L1, L2 = np.zeros((K, r), np.int8), np.zeros((r, N), np.int8)
        sL1, sL2 = np.zeros(r, np.float32), np.zeros(N, np.float32)
    _check(lib().lq_layer_export(layer, _np_ptr(out["Wq_packed"]), _np_ptr(out["sw"]), _np_ptr(L1), _np_ptr(sL1),
                                 _np_ptr(L2), _np_ptr(sL2), _np_ptr(out["bias"])), "lq_layer_export")
    out.update(L1=L1, L2=L2, sL1=sL1, sL2=sL2)
    return out


def lq_layer_to_device(layer, device: int = 0):
    _check(lib().lq_layer_to_device(layer, device), "lq_layer_to_device")


def lq_layer_free(layer):
    _check(lib().lq_layer_free(layer), "lq_layer_free")


def lq_act_create(layer, M_max: int, device: int = 0):
    h = C.c_void_p()
    _check(lib().lq_act_create(layer, M_max, device, C.byref(h)), "lq_act_create")
    return h


def lq_act_free(act):
    _check(lib().lq_act_free(act), "lq_act_free")


def lq_quantize_act(layer, X_dev_ptr: int, M: int, act, stream: int = 0):
    _check(lib().lq_quantize_act(layer, C.c_void_p(X_dev_ptr), M, act, C.c_void_p(stream)), "lq_quantize_act")


def lq_linear_forward(layer, act, Y_dev_ptr: int, dtype: int = OUT_F16, stream: int = 0):
    _check(lib().lq_linear_forward(layer, act, C.c_void_p(Y_dev_ptr), dtype, C.c_void_p(stream)), "lq_linear_forward")


def lq_linear_forward_host(layer, act, X_host_ptr: int, M: int, Y_host_ptr: int, dtype: int = OUT_F16, stream: int = 0):
    _check(lib().lq_linear_forward_host(layer, act, C.c_void_p(X_host_ptr), M, C.c_void_p(Y_host_ptr), dtype,
                                        C.c_void_p(stream)), "lq_linear_forward_host")


def lq_linear_forward_host_async(layer, act, X_host_ptr: int, M: int, Y_host_ptr: int, dtype: int = OUT_F16, stream: int = 0):
    _check(lib().lq_linear_forward_host_async(layer, act, C.c_void_p(X_host_ptr), M, C.c_void_p(Y_host_ptr), dtype,
                                        C.c_void_p(stream)), "lq_linear_forward_host_async")


STATIC_SCRATCH_BYTES = 8 << 20


def lq_linear_forward_static(layer, X_dev_ptr: int, M: int, Y_dev_ptr: int, dtype: int = OUT_F16, stream: int = 0):
    """Whole forward without any allocation at call time: the activation record lives in a fixed
    device array inside the library (for callers whose memory pool forbids raw allocations).
    Raises LqError(code 2) when M x K does not fit the array; calls must not overlap on the GPU."""
    _check(lib().lq_linear_forward_static(layer, C.c_void_p(X_dev_ptr), M, C.c_void_p(Y_dev_ptr), dtype,
                                          C.c_void_p(stream)), "lq_linear_forward_static")


def lq_act_export(act, M: int, cfg: LqConfig, stream: int = 0) -> dict:
    K, r, G = cfg.K, cfg.rank, -(-cfg.K // cfg.group)
    if cfg.main_fmt in (MAIN_MXFP4, MAIN_MXINT4_A8):
        # MXFP: qx / tq are e4m3 bit patterns (decode with e4m3_decode); integer MX with 8-bit activations: the int8 codes.
        # sx: the int16 block exponents of X; sT: the block exponents of the rank-r intermediate as floats [M, ceil(r/32)]
        out = {"qx": np.zeros((M, K), np.int8), "sx": np.zeros((M, G), np.int16), "qb": None, "sXb": None, "tq": None, "sT": None}
        if r > 0 and cfg.branch != BRANCH["none"]:
            out["tq"] = np.zeros((M, r), np.int8)
            out["sT"] = np.zeros((M, -(-r // 32)), np.float32)
        _check(lib().lq_act_export(act, _np_ptr(out["qx"]), _np_ptr(out["sx"]), None, None, _np_ptr(out["tq"]),
                                   _np_ptr(out["sT"]), C.c_void_p(stream)), "lq_act_export")
        return out
    # SINT4: fp16 group scales; MXINT4 (group 32): int16 block exponents e (scale 2^e)
    out = {"qx": np.zeros((M, K), np.int8), "sx": np.zeros((M, G), np.int16 if cfg.group == 32 else np.float16)}
    qb = sXb = tq = sT = None
    if r > 0 and cfg.branch != BRANCH["none"]:
        f16 = cfg.branch == BRANCH["w16a16"]
        tq = np.zeros((M, r), np.float16 if f16 else np.int8)
        sT = np.zeros(M, np.float32)
        if not f16:
            qb, sXb = np.zeros((M, K), np.int8), np.zeros(M, np.float32)
    _check(lib().lq_act_export(act, _np_ptr(out["qx"]), _np_ptr(out["sx"]), _np_ptr(qb), _np_ptr(sXb), _np_ptr(tq),
                               _np_ptr(sT), C.c_void_p(stream)), "lq_act_export")
    out.update(qb=qb, sXb=sXb, tq=tq, sT=sT)
    return out


def lq_get_device_status(device: int = 0):
    code, stage = C.c_int32(), C.c_int32()
    _check(lib().lq_get_device_status(device, C.byref(code), C.byref(stage)), "lq_get_device_status")
    return code.value, stage.value


def lq_selftest_wait_timeout(device: int = 0, stream: int = 0):
    _check(lib().lq_selftest_wait_timeout(device, C.c_void_p(stream)), "lq_selftest_wait_timeout")


def lq_set_option(name: str, value: int):
    _check(lib().lq_set_option(name.encode(), value), "lq_set_option")


def lq_version() -> int:
    return lib().lq_version()
