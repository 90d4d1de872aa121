"""Thin ctypes binding over libhq.so: same names as the C ABI, argument marshalling only.

torch is used for device memory and streams; every step of the inference path runs inside the
library's CUDA kernels.  There is no CPU fallback: if the shared library is missing or the device
is not a B200-class GPU, loading or hq_create fails loudly.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libhq.so")

HQ_OK, HQ_ERR_INVALID_ARG, HQ_ERR_UNSUPPORTED, HQ_ERR_ALIGNMENT = 0, 1, 2, 3
HQ_ERR_RANGE, HQ_ERR_WORKSPACE, HQ_ERR_CUDA, HQ_ERR_TIMEOUT, HQ_ERR_INFEASIBLE = 4, 5, 6, 7, 8
HQ_OP = {"conv": 0, "linear": 1, "maxpool": 2, "avgpool": 3, "add": 4, "requant": 5, "concat": 6, "sumpool": 7}

EXPORTS = [
    "hq_create", "hq_destroy", "hq_sync", "hq_conv2d", "hq_linear", "hq_residual_add", "hq_avgpool_requant",
    "hq_maxpool", "hq_network_create", "hq_run_network", "hq_network_layer_bytes", "hq_network_launch_count",
    "hq_network_destroy", "hq_set_conv_path", "hq_set_tile_order", "hq_status_string", "hq_network_time_layers", "hq_conv2d_noalloc", "hq_expire_wait_selftest",
    "hq_network_check_guards", "hq_conv2d_noalloc_sync", "hq_mma_peak_launch",
    "hq_ilp_solve", "hq_concat_requant", "hq_sumpool",
]


class HqError(RuntimeError):
    def __init__(self, code: int, where: str):
        super().__init__(f"{where}: {status_string(code)} ({code})")
        self.code = code


class hq_tensor(C.Structure):
    _fields_ = [("data", C.c_void_p), ("n", C.c_int32), ("h", C.c_int32), ("w", C.c_int32), ("c", C.c_int32),
                ("bits", C.c_int32), ("is_signed", C.c_int32)]


class hq_dyadic(C.Structure):
    _fields_ = [("b", C.c_void_p), ("c", C.c_void_p)]


class hq_conv_desc(C.Structure):
    _fields_ = [("kh", C.c_int32), ("kw", C.c_int32), ("stride", C.c_int32), ("pad", C.c_int32),
                ("cin", C.c_int32), ("cout", C.c_int32), ("w_bits", C.c_int32), ("w", C.c_void_p),
                ("bias", C.c_void_p), ("requant", hq_dyadic), ("residual", C.POINTER(hq_tensor)),
                ("res_rescale", hq_dyadic), ("relu", C.c_int32), ("qmin", C.c_int32), ("qmax", C.c_int32)]


class hq_layer(C.Structure):
    _fields_ = [("op", C.c_int32), ("in0", C.c_int32), ("in1", C.c_int32), ("conv", hq_conv_desc),
                ("rescale0", hq_dyadic), ("rescale1", hq_dyadic), ("pool_k", C.c_int32),
                ("pool_stride", C.c_int32), ("pool_pad", C.c_int32), ("out_bits", C.c_int32),
                ("out_signed", C.c_int32), ("relu", C.c_int32), ("qmin", C.c_int32), ("qmax", C.c_int32),
                ("n_in", C.c_int32), ("ins", C.c_int32 * 8), ("rescales", hq_dyadic * 8)]


_lib = None


def lib():
    """Load libhq.so (must have been built in-tree; see build.py)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build the CUDA library first (python -m paper_2011_10680_b200.build)")
        L = C.CDLL(LIB_PATH)
        vp, i32 = C.c_void_p, C.c_int32
        TP, DP, LP = C.POINTER(hq_tensor), C.POINTER(hq_conv_desc), C.POINTER(hq_layer)
        L.hq_create.argtypes = [i32, C.POINTER(vp)]
        L.hq_destroy.argtypes = [vp]
        L.hq_sync.argtypes = [vp, vp]
        L.hq_conv2d.argtypes = [vp, TP, DP, TP, vp]
        L.hq_linear.argtypes = [vp, TP, DP, TP, vp]
        L.hq_residual_add.argtypes = [vp, TP, hq_dyadic, TP, hq_dyadic, i32, i32, i32, TP, vp]
        L.hq_avgpool_requant.argtypes = [vp, TP, hq_dyadic, i32, i32, TP, vp]
        L.hq_maxpool.argtypes = [vp, TP, i32, i32, i32, TP, vp]
        L.hq_sumpool.argtypes = [vp, TP, i32, i32, i32, TP, vp]
        L.hq_concat_requant.argtypes = [vp, i32, TP, C.POINTER(hq_dyadic), i32, i32, i32, TP, vp]
        L.hq_network_create.argtypes = [vp, LP, i32, i32, i32, i32, i32, i32, C.POINTER(vp)]
        L.hq_run_network.argtypes = [vp, TP, TP, C.POINTER(vp), vp]
        L.hq_conv2d_noalloc.argtypes = [TP, DP, TP, vp]
        L.hq_network_time_layers.argtypes = [vp, TP, TP, C.POINTER(C.c_int64), vp]
        L.hq_network_layer_bytes.argtypes = [vp, i32, C.POINTER(C.c_int64)]
        L.hq_network_launch_count.argtypes = [vp, C.POINTER(i32)]
        L.hq_network_destroy.argtypes = [vp]
        L.hq_network_check_guards.argtypes = [vp, vp, C.POINTER(i32)]
        L.hq_conv2d_noalloc_sync.argtypes = [vp]
        L.hq_mma_peak_launch.argtypes = [vp, i32, i32, C.POINTER(C.c_int64), vp]
        L.hq_set_conv_path.argtypes = [vp, i32]
        L.hq_set_tile_order.argtypes = [vp, i32]
        L.hq_expire_wait_selftest.argtypes = [vp, i32, vp]
        L.hq_expire_wait_selftest.restype = i32
        i64p = C.POINTER(C.c_int64)
        L.hq_ilp_solve.argtypes = [i32, i64p, i64p, i64p, i64p, C.c_int64, C.c_int64, C.c_int64, C.POINTER(i32), i64p]
        L.hq_status_string.argtypes = [i32]
        L.hq_status_string.restype = C.c_char_p
        for name in EXPORTS:
            if name != "hq_status_string":
                getattr(L, name).restype = i32
        _lib = L
    return _lib


def ilp_solve(omega, size, bops, latency, size_limit: int = -1, bops_limit: int = -1, latency_limit: int = -1):
    """hq_ilp_solve on host arrays of shape [n_layers, 2] (int64).  Returns (status, choices, objective)."""
    tabs = [np.ascontiguousarray(t, dtype=np.int64) for t in (omega, size, bops, latency)]
    n = tabs[0].shape[0]
    if any(t.shape != (n, 2) for t in tabs):
        raise ValueError("every table must have shape [n_layers, 2]")
    choice = np.zeros(max(n, 1), dtype=np.int32)
    obj = C.c_int64(0)
    i64p = C.POINTER(C.c_int64)
    st = lib().hq_ilp_solve(n, *[t.ctypes.data_as(i64p) for t in tabs], int(size_limit), int(bops_limit),
                            int(latency_limit), choice.ctypes.data_as(C.POINTER(C.c_int32)), C.byref(obj))
    return st, choice[:n].copy(), int(obj.value)


def status_string(code: int) -> str:
    return lib().hq_status_string(code).decode()


def _check(code: int, where: str):
    if code != HQ_OK:
        raise HqError(code, where)


def _stream():
    import torch
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def tensor_of(t, c: int, bits: int, is_signed: int) -> hq_tensor:
    """Describe a torch CUDA tensor of shape (n, h, w, c_stored) as an hq_tensor with logical channels c."""
    n, h, w = t.shape[0], t.shape[1], t.shape[2]
    return hq_tensor(t.data_ptr(), n, h, w, c, bits, is_signed)


def _dy(b, c) -> hq_dyadic:
    return hq_dyadic(b.data_ptr() if b is not None else None, c.data_ptr() if c is not None else None)


def to_device(a):
    """numpy array -> CUDA tensor with the same bytes (int8/uint8/int32)."""
    import torch
    if a is None:
        return None
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


GUARD_BYTES, GUARD_VALUE = 4096, 0xA5
_guarded = []          # (flat uint8 buffer, payload bytes) of every output handed out since the last check


def alloc_out(n, h, w, c, bits, signed):
    """Output tensor of a call, allocated between two 4 KiB guard bands filled with 0xA5 (the stand-in for a
    memory checker: check_guards() finds any byte a kernel wrote before the first or after the last element)."""
    import torch
    dtype = torch.int32 if bits == 32 else (torch.int8 if (bits == 8 and signed) else torch.uint8)
    shape = (n, h, w, c // 2) if bits == 4 else (n, h, w, c)
    nbytes = n * h * w * c * bits // 8
    flat = torch.empty(nbytes + 2 * GUARD_BYTES, dtype=torch.uint8, device="cuda")
    flat[:GUARD_BYTES] = GUARD_VALUE
    flat[GUARD_BYTES + nbytes:] = GUARD_VALUE
    _guarded.append((flat, nbytes))
    return flat[GUARD_BYTES:GUARD_BYTES + nbytes].view(dtype).view(shape)


def check_guards():
    """Verify (and forget) the guard bands of every tensor alloc_out returned; raises on a touched byte."""
    import torch
    torch.cuda.synchronize()
    bad = []
    for flat, nbytes in _guarded:
        lo, hi = flat[:GUARD_BYTES], flat[GUARD_BYTES + nbytes:]
        if not (bool((lo == GUARD_VALUE).all()) and bool((hi == GUARD_VALUE).all())):
            before = int((lo != GUARD_VALUE).sum())
            after = int((hi != GUARD_VALUE).sum())
            bad.append(f"{nbytes}-byte output: {before} bytes written before it, {after} after it")
    _guarded.clear()
    if bad:
        raise AssertionError("a kernel wrote outside its output tensor: " + "; ".join(bad))


class Handle:
    """Owns an hq_handle for one device."""

    def __init__(self, device: int = 0):
        self._h = C.c_void_p()
        _check(lib().hq_create(device, C.byref(self._h)), "hq_create")

    def close(self):
        if self._h:
            lib().hq_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def set_conv_path(self, path: int):
        _check(lib().hq_set_conv_path(self._h, path), "hq_set_conv_path")

    def set_tile_order(self, order: int):
        _check(lib().hq_set_tile_order(self._h, order), "hq_set_tile_order")

    def expire_wait_selftest(self, budget_ms: int) -> int:
        return lib().hq_expire_wait_selftest(self._h, budget_ms, _stream())

    def sync(self):
        _check(lib().hq_sync(self._h, _stream()), "hq_sync")

    def mma_peak_launch(self, rounds: int, blocks_per_round: int) -> int:
        """hq_mma_peak_launch on the current stream; returns the integer operations the launch performs."""
        ops = C.c_int64()
        _check(lib().hq_mma_peak_launch(self._h, rounds, blocks_per_round, C.byref(ops), _stream()), "hq_mma_peak_launch")
        return ops.value

    # ---- one call per C entry point --------------------------------------------------------
    def conv2d(self, x, in_bits, in_signed, cin, wgt, cout, kh, kw, stride, pad, bias, b, c, out, out_bits, out_signed,
               res=None, res_bits=0, res_signed=0, rb=None, rc=None, relu=1, qmin=0, qmax=255, linear=False):
        tin = tensor_of(x, cin, in_bits, in_signed)
        tout = tensor_of(out, cout, out_bits, out_signed)
        tres = tensor_of(res, cout, res_bits, res_signed) if res is not None else None
        d = hq_conv_desc(kh, kw, stride, pad, cin, cout, in_bits, wgt.data_ptr(),
                         bias.data_ptr() if bias is not None else None, _dy(b, c),
                         C.pointer(tres) if tres is not None else None, _dy(rb, rc), relu, qmin, qmax)
        fn = lib().hq_linear if linear else lib().hq_conv2d
        return fn(self._h, C.byref(tin), C.byref(d), C.byref(tout), _stream())

    def residual_add(self, main, main_bits, main_signed, mb, mc, res, res_bits, res_signed, rb, rc, ch,
                     relu, qmin, qmax, out, out_bits, out_signed):
        tm = tensor_of(main, ch, main_bits, main_signed)
        to = tensor_of(out, ch, out_bits, out_signed)
        tr = tensor_of(res, ch, res_bits, res_signed) if res is not None else None
        return lib().hq_residual_add(self._h, C.byref(tm), _dy(mb, mc), C.byref(tr) if tr is not None else None,
                                     _dy(rb, rc), relu, qmin, qmax, C.byref(to), _stream())

    def avgpool_requant(self, x, ch, in_bits, in_signed, b, c, qmin, qmax, out, out_bits, out_signed):
        ti = tensor_of(x, ch, in_bits, in_signed)
        to = tensor_of(out, ch, out_bits, out_signed)
        return lib().hq_avgpool_requant(self._h, C.byref(ti), _dy(b, c), qmin, qmax, C.byref(to), _stream())

    def concat_requant(self, branches, relu, qmin, qmax, out, out_bits, out_signed):
        """`branches`: list of dicts {x, bits, signed, ch, b, c} of CUDA tensors; `out`: (n, h, w, sum ch)."""
        n = len(branches)
        ts = (hq_tensor * n)(*[tensor_of(br["x"], br["ch"], br["bits"], br["signed"]) for br in branches])
        ds = (hq_dyadic * n)(*[_dy(br["b"], br["c"]) for br in branches])
        to = tensor_of(out, out.shape[3] * (2 if out_bits == 4 else 1), out_bits, out_signed)
        return lib().hq_concat_requant(self._h, n, ts, ds, relu, qmin, qmax, C.byref(to), _stream())

    def sumpool(self, x, ch, bits, signed, k, stride, pad, out):
        ti = tensor_of(x, ch, bits, signed)
        to = tensor_of(out, ch, 32, 1)
        return lib().hq_sumpool(self._h, C.byref(ti), k, stride, pad, C.byref(to), _stream())

    def maxpool(self, x, ch, signed, k, stride, pad, out, bits: int = 8):
        ti = tensor_of(x, ch, bits, signed)
        to = tensor_of(out, ch, bits, signed)
        return lib().hq_maxpool(self._h, C.byref(ti), k, stride, pad, C.byref(to), _stream())

    # ---- convenience for the dict-shaped single-layer cases of the workload generator -------
    def conv_case(self, case: dict, dev: dict | None = None, out=None):
        """Upload (or reuse `dev`) a generated conv case, run hq_conv2d, return (status, out tensor).  `out`: an output
        tensor allocated by the caller (a timing loop keeps the allocation and its guard-band fills out of the timed region)."""
        dev = dev if dev is not None else upload_case(case)
        if out is None:
            out = alloc_out(case["n"], case["ho"], case["wo"], case["cout"], case["out_bits"], case["out_signed"])
        st = self.conv2d(dev["x"], case["bits"], case["in_signed"], case["cin"], dev["wgt"], case["cout"], case["kh"],
                         case["kw"], case["stride"], case["pad"], dev["bias"], dev["b"], dev["c"], out,
                         case["out_bits"], case["out_signed"], dev["res"], case["res_bits"], case["res_signed"],
                         dev["rb"], dev["rc"], case["relu"], case["qmin"], case["qmax"])
        return st, out


def conv2d_noalloc(case: dict, dev: dict, out):
    """hq_conv2d_noalloc on an uploaded conv case: no handle, no allocation inside the library."""
    tin = tensor_of(dev["x"], case["cin"], case["bits"], case["in_signed"])
    tout = tensor_of(out, case["cout"], case["out_bits"], case["out_signed"])
    tres = tensor_of(dev["res"], case["cout"], case["res_bits"], case["res_signed"]) if dev["res"] is not None else None
    d = hq_conv_desc(case["kh"], case["kw"], case["stride"], case["pad"], case["cin"], case["cout"], case["bits"],
                     dev["wgt"].data_ptr(), dev["bias"].data_ptr() if dev["bias"] is not None else None,
                     _dy(dev["b"], dev["c"]), C.pointer(tres) if tres is not None else None, _dy(dev["rb"], dev["rc"]),
                     case["relu"], case["qmin"], case["qmax"])
    return lib().hq_conv2d_noalloc(C.byref(tin), C.byref(d), C.byref(tout), _stream())


def conv2d_noalloc_sync() -> int:
    return lib().hq_conv2d_noalloc_sync(_stream())


def upload_case(case: dict) -> dict:
    return {k: to_device(case[k]) for k in ("x", "wgt", "bias", "b", "c", "res", "rb", "rc")}


class Network:
    """hq_network built from a generated layer table; keeps the device copies of all parameters alive."""

    def __init__(self, handle: Handle, table: dict, batch: int, image_signed: int = 0):
        self.handle, self.table, self.batch = handle, table, batch
        self._keep = []
        layers = table["layers"]
        arr = (hq_layer * len(layers))()
        for i, l in enumerate(layers):
            e = arr[i]
            e.op, e.in0, e.in1 = HQ_OP[l["op"]], l["in0"], l["in1"]
            e.out_bits, e.out_signed = l["out_bits"], l["out_signed"]
            e.relu, e.qmin, e.qmax = l["relu"], l["qmin"], l["qmax"]
            if l["op"] in ("conv", "linear"):
                dv = {k: to_device(l[k]) for k in ("wgt", "bias", "b", "c", "rb", "rc")}
                self._keep.append(dv)
                e.conv = hq_conv_desc(l["kh"], l["kw"], l["stride"], l["pad"], l["cin"], l["cout"], l["bits"],
                                      dv["wgt"].data_ptr(),
                                      dv["bias"].data_ptr() if dv["bias"] is not None else None, _dy(dv["b"], dv["c"]), None,
                                      _dy(dv["rb"], dv["rc"]), l["relu"], l["qmin"], l["qmax"])
            elif l["op"] in ("maxpool", "sumpool"):
                e.pool_k, e.pool_stride, e.pool_pad = l["pool_k"], l["pool_stride"], l["pool_pad"]
            elif l["op"] == "concat":
                e.n_in, e.in0 = len(l["ins"]), l["ins"][0]
                for k, (tid, b, c) in enumerate(zip(l["ins"], l["bs"], l["cs"])):
                    dv = {"b": to_device(b), "c": to_device(c)}
                    self._keep.append(dv)
                    e.ins[k] = tid
                    e.rescales[k] = _dy(dv["b"], dv["c"])
            else:
                dv = {k: to_device(l.get(k)) for k in ("b", "c", "rb", "rc")}
                self._keep.append(dv)
                e.rescale0 = _dy(dv["b"], dv["c"])
                e.rescale1 = _dy(dv["rb"], dv["rc"])
        self._arr = arr
        self._net = C.c_void_p()
        hw = table["image_hw"]
        _check(lib().hq_network_create(handle._h, arr, len(layers), batch, hw, hw, 3, image_signed,
                                       C.byref(self._net)), "hq_network_create")
        last = layers[-1]
        self.logits_shape = (batch, 1, 1, last["cout"])

    def layer_bytes(self, i: int) -> int:
        v = C.c_int64()
        _check(lib().hq_network_layer_bytes(self._net, i, C.byref(v)), "hq_network_layer_bytes")
        return v.value

    def launch_count(self) -> int:
        v = C.c_int32()
        _check(lib().hq_network_launch_count(self._net, C.byref(v)), "hq_network_launch_count")
        return v.value

    def run(self, images, logits, taps=None):
        """images: uint8 CUDA tensor (batch, H, W, 3); logits: int32 CUDA tensor; taps: list of CUDA tensors or None."""
        ti = tensor_of(images, images.shape[3], 8, 0)
        last = self.table["layers"][-1]
        tl = hq_tensor(logits.data_ptr(), self.batch, 1, 1, last["cout"], last["out_bits"], last["out_signed"])
        tap_arr = None
        if taps is not None:
            tap_arr = (C.c_void_p * len(taps))(*[t.data_ptr() if t is not None else None for t in taps])
        return lib().hq_run_network(self._net, C.byref(ti), C.byref(tl), tap_arr, _stream())

    def time_layers(self, images, logits):
        """Per-layer device time in nanoseconds (CUDA events around each layer, plain launches)."""
        ti = tensor_of(images, images.shape[3], 8, 0)
        last = self.table["layers"][-1]
        tl = hq_tensor(logits.data_ptr(), self.batch, 1, 1, last["cout"], last["out_bits"], last["out_signed"])
        ns = (C.c_int64 * len(self.table["layers"]))()
        _check(lib().hq_network_time_layers(self._net, C.byref(ti), C.byref(tl), ns, _stream()), "hq_network_time_layers")
        return list(ns)

    def alloc_taps(self):
        return [alloc_out(1, 1, 1, self.layer_bytes(i), 8, 0).view(-1) for i in range(len(self.table["layers"]))]

    def check_guards(self):
        """hq_network_check_guards: raises if a kernel wrote outside one of the network's own buffers."""
        bad = C.c_int32(-2)
        st = lib().hq_network_check_guards(self._net, _stream(), C.byref(bad))
        if st != HQ_OK:
            raise AssertionError(f"hq_network_check_guards: {status_string(st)}, buffer of layer {bad.value}")

    def close(self):
        if self._net:
            lib().hq_network_destroy(self._net)
            self._net = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
