"""ctypes binding of libexmoe.so: the same entry points as include/exmoe.h, argument marshalling only.

PyTorch provides device memory, pinned host memory and streams; every step of the layer runs in
the library's own CUDA kernels.  There is no fallback: if the library is missing or a call fails,
an exception is raised.
"""
import ctypes
import os
from ctypes import POINTER, byref, c_char_p, c_float, c_int, c_int32, c_size_t, c_uint64, c_void_p

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libexmoe.so")

EXMOE_OK = 0
EXMOE_ERR_ARG = -1
EXMOE_ERR_SHAPE = -2
EXMOE_ERR_NOT_PINNED = -3
EXMOE_ERR_CUDA = -4
EXMOE_ERR_NONFINITE = -5
EXMOE_ERR_BAD_EXPERT_ID = -6
EXMOE_ERR_TIMEOUT = -7
EXMOE_ERR_STATE = -8


class ExmoeError(RuntimeError):
    def __init__(self, code, what):
        self.code = code
        super().__init__(f"{what}: {strerror(code)} ({code})")


class exmoe_shape(ctypes.Structure):
    _fields_ = [("d_model", c_int), ("d_ff", c_int), ("num_experts", c_int), ("top_k", c_int), ("group_size", c_int)]


class exmoe_stats(ctypes.Structure):
    _fields_ = [("lookups", c_uint64), ("hits", c_uint64), ("misses", c_uint64), ("waves", c_uint64),
                ("h2d_bytes", c_uint64), ("forwards", c_uint64)]


_SIGNATURES = {
    "exmoe_strerror": (c_char_p, [c_int]),
    "exmoe_packed_bytes": (c_int, [POINTER(exmoe_shape), POINTER(c_size_t)]),
    "exmoe_pack": (c_int, [POINTER(exmoe_shape), c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]),
    "exmoe_cache_workspace_bytes": (c_int, [POINTER(exmoe_shape), c_int, c_int, c_int, POINTER(c_size_t), POINTER(c_size_t)]),
    "exmoe_cache_create": (c_int, [POINTER(c_void_p), POINTER(exmoe_shape), c_int, c_int, POINTER(c_void_p), c_void_p,
                                   c_void_p, c_int, c_int]),
    "exmoe_moe_forward": (c_int, [c_void_p, c_int, c_void_p, c_void_p, c_void_p, c_int, c_void_p, c_void_p]),
    "exmoe_moe_forward_host": (c_int, [c_void_p, c_int, c_void_p, c_void_p, c_void_p, c_int, c_void_p, c_void_p]),
    "exmoe_moe_forward_static_status": (c_int, []),
    "exmoe_debug_last_host_copy_bytes": (c_int, [c_void_p, POINTER(c_size_t)]),
    "exmoe_moe_forward_static": (c_int, [POINTER(exmoe_shape), c_void_p, c_void_p, c_void_p, c_void_p, c_int, c_void_p, c_void_p]),
    "exmoe_route": (c_int, [POINTER(exmoe_shape), c_void_p, c_void_p, c_void_p, c_int, c_void_p, c_void_p, c_void_p]),
    "exmoe_cache_get_state": (c_int, [c_void_p, c_int, c_void_p, c_void_p, c_void_p, c_void_p]),
    "exmoe_debug_last_plan": (c_int, [c_void_p, c_int] + [c_void_p] * 9),
    "exmoe_debug_last_path": (c_int, [c_void_p]),
    "exmoe_debug_read_slot": (c_int, [c_void_p, c_int, c_int, c_void_p]),
    "exmoe_debug_wait_timeout": (c_int, [c_void_p, ctypes.c_longlong, POINTER(c_int)]),
    "exmoe_cache_stats": (c_int, [c_void_p, c_int, POINTER(exmoe_stats)]),
    "exmoe_cache_reset": (c_int, [c_void_p, c_int]),
    "exmoe_cache_set_miss_path": (c_int, [c_void_p, c_int]),
    "exmoe_cache_prefetch": (c_int, [c_void_p, c_int, c_void_p, c_int, c_void_p]),
    "exmoe_status": (c_int, [c_void_p]),
    "exmoe_cache_destroy": (c_int, [c_void_p]),
    "exmoe_profile_enable": (c_int, [c_void_p, c_int]),
    "exmoe_profile_read": (c_int, [c_void_p, c_int, POINTER(ctypes.c_double), POINTER(c_uint64)]),
    "exmoe_profile_overlap": (c_int, [c_void_p, POINTER(ctypes.c_double), POINTER(ctypes.c_double)]),
    "exmoe_launch_count": (c_uint64, []),
}

_lib = None


def lib():
    """Open libexmoe.so (built in-tree by `paper_2608_15383_b200.build`); fail loudly if absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise FileNotFoundError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2608_15383_b200.build` (no CPU fallback exists)")
        h = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in _SIGNATURES.items():
            fn = getattr(h, name)
            fn.restype = res
            fn.argtypes = args
        _lib = h
    return _lib


def strerror(code):
    return lib().exmoe_strerror(int(code)).decode()


def _check(code, what):
    if code != EXMOE_OK:
        raise ExmoeError(code, what)


def _shape(s):
    return exmoe_shape(int(s.d_model), int(s.d_ff), int(s.num_experts), int(s.top_k), int(getattr(s, "group_size", 128)))


def _stream_ptr(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return c_void_p(stream.cuda_stream)


def _dev(t, dtype, what):
    if not (t.is_cuda and t.dtype == dtype and t.is_contiguous()):
        raise ValueError(f"{what}: need a contiguous CUDA tensor of {dtype}")
    return c_void_p(t.data_ptr())


# ------------------------------------------------------------------------------------ C names
def exmoe_packed_bytes(shape):
    n = c_size_t()
    _check(lib().exmoe_packed_bytes(byref(_shape(shape)), byref(n)), "exmoe_packed_bytes")
    return n.value


def exmoe_pack(shape, w_gate, w_up, w_down, packed_out=None, stream=None):
    """Quantise and pack ONE expert on the GPU.  Returns the packed uint8 tensor (device)."""
    I, H = shape.d_ff, shape.d_model
    if tuple(w_gate.shape) != (I, H) or tuple(w_up.shape) != (I, H) or tuple(w_down.shape) != (H, I):
        raise ValueError("exmoe_pack: weight shapes must be [I,H], [I,H], [H,I]")
    if packed_out is None:
        packed_out = torch.empty(exmoe_packed_bytes(shape), dtype=torch.uint8, device=w_gate.device)
    rc = lib().exmoe_pack(byref(_shape(shape)), _dev(w_gate, torch.bfloat16, "w_gate"),
                          _dev(w_up, torch.bfloat16, "w_up"), _dev(w_down, torch.bfloat16, "w_down"),
                          _dev(packed_out, torch.uint8, "packed_out"), _stream_ptr(stream))
    _check(rc, "exmoe_pack")
    return packed_out


def exmoe_cache_workspace_bytes(shape, num_layers, num_slots, max_tokens):
    a, b = c_size_t(), c_size_t()
    _check(lib().exmoe_cache_workspace_bytes(byref(_shape(shape)), num_layers, num_slots, max_tokens, byref(a), byref(b)),
           "exmoe_cache_workspace_bytes")
    return a.value, b.value


def exmoe_moe_forward_static(shape, experts_dev, hidden, topk_ids, topk_weights, out, stream=None):
    """Tiny-batch forward through the library's built-in scratch: no cache object, no workspace, nothing is
    allocated by the call (the caller passes `out`).  For callers that cannot obtain device memory when they
    need the layer; limits: T * top_k <= 32, d_ff <= 4096, fully resident experts."""
    rc = lib().exmoe_moe_forward_static(byref(_shape(shape)), _dev(experts_dev, torch.uint8, "experts_dev"),
                                        _dev(hidden, torch.bfloat16, "hidden"), _dev(topk_ids, torch.int32, "topk_ids"),
                                        _dev(topk_weights, torch.float32, "topk_weights"), int(hidden.shape[0]),
                                        _dev(out, torch.bfloat16, "out"), _stream_ptr(stream))
    _check(rc, "exmoe_moe_forward_static")
    return out


def exmoe_moe_forward_static_status():
    """Sticky device-side status of exmoe_moe_forward_static on the current device (synchronises, clears)."""
    return int(lib().exmoe_moe_forward_static_status())


def exmoe_route(shape, hidden, w_router, bias=None, topk_ids=None, topk_weights=None, stream=None):
    """Eq. 1 on the device: logits, softmax over all experts, top-k.  Returns (ids int32 [T, k], weights fp32 [T, k])."""
    T = int(hidden.shape[0])
    if topk_ids is None:
        topk_ids = torch.empty((T, shape.top_k), dtype=torch.int32, device=hidden.device)
    if topk_weights is None:
        topk_weights = torch.empty((T, shape.top_k), dtype=torch.float32, device=hidden.device)
    rc = lib().exmoe_route(byref(_shape(shape)), _dev(hidden, torch.bfloat16, "hidden"),
                           _dev(w_router, torch.bfloat16, "w_router"),
                           _dev(bias, torch.float32, "bias") if bias is not None else None, T,
                           _dev(topk_ids, torch.int32, "topk_ids"), _dev(topk_weights, torch.float32, "topk_weights"),
                           _stream_ptr(stream))
    _check(rc, "exmoe_route")
    return topk_ids, topk_weights


def exmoe_launch_count():
    return int(lib().exmoe_launch_count())


def pack_bank(shape, w_gate, w_up, w_down, device="cuda"):
    """Pack all experts of one layer ([E,I,H], [E,I,H], [E,H,I] BF16) into a pinned host bank [E, bytes]."""
    E = shape.num_experts
    n = exmoe_packed_bytes(shape)
    bank = torch.empty((E, n), dtype=torch.uint8).pin_memory()
    buf = torch.empty(n, dtype=torch.uint8, device=device)
    for e in range(E):
        exmoe_pack(shape, w_gate[e].to(device).contiguous(), w_up[e].to(device).contiguous(),
                   w_down[e].to(device).contiguous(), buf)
        bank[e].copy_(buf)
    return bank


def padded_dims(d_model, d_ff, group=128):
    """Section 3.2 asks for dims that are multiples of the group size and Section 7 leaves other shapes to padding: the
    next multiples of 128."""
    up = lambda n: -(-int(n) // group) * group
    return up(d_model), up(d_ff)


def pad_expert_weights(w_gate, w_up, w_down, group=128):
    """Zero-pad [E, I, H], [E, I, H], [E, H, I] expert tensors to multiples of 128 in both dims.  The padded
    intermediate channels compute SiLU(0) * 0 = 0 and meet zero columns of W_down; the padded hidden channels meet
    zero weights: columns [0, H) of the padded layer's output are the layer applied to the unpadded hidden state
    (quantised in groups that end at the padded length), columns [H, H_pad) are zero.  Pad the hidden state with
    pad_hidden and slice the output back."""
    E, I, H = w_gate.shape
    Hp, Ip = padded_dims(H, I, group)
    pad = torch.nn.functional.pad
    return (pad(w_gate, (0, Hp - H, 0, Ip - I)).contiguous(), pad(w_up, (0, Hp - H, 0, Ip - I)).contiguous(),
            pad(w_down, (0, Ip - I, 0, Hp - H)).contiguous())


def pad_hidden(hidden, d_model_padded):
    return torch.nn.functional.pad(hidden, (0, d_model_padded - hidden.shape[-1])).contiguous()


MISS_HOST_COPIES, MISS_DEVICE_FETCH = 0, 1
PATH_PAIR, PATH_SMALL, PATH_STREAM, PATH_TENSOR_SMALL_N, PATH_TENSOR = 2, 3, 4, 5, 6


class Cache:
    """exmoe_cache handle plus the torch buffers it borrows (slot memory, workspace, host banks)."""

    GUARD_BYTE = 0xA5

    def __init__(self, shape, banks, num_slots, max_tokens, wave_cap=0, device="cuda", guard_bytes=0):
        """guard_bytes > 0 (a multiple of 256): slot memory and workspace are carved out of larger tensors whose
        margins on both sides are filled with GUARD_BYTE; guards_intact() tells whether any kernel wrote there."""
        self.shape, self.C, self.L = shape, int(num_slots), len(banks)
        self.max_tokens = int(max_tokens)
        self.wave_cap = int(wave_cap) if wave_cap else int(num_slots)
        self.bytes_per_expert = exmoe_packed_bytes(shape)
        slot_bytes, ws_bytes = exmoe_cache_workspace_bytes(shape, self.L, self.C, self.max_tokens)
        self.banks = list(banks)
        g = int(guard_bytes)
        if g % 256:
            raise ValueError("guard_bytes must be a multiple of 256")
        self._guarded = []
        bufs = []
        for n in (slot_bytes, ws_bytes):
            n_al = -(-n // 256) * 256
            whole = torch.full((n_al + 2 * g,), self.GUARD_BYTE, dtype=torch.uint8, device=device) if g else \
                torch.empty(n_al, dtype=torch.uint8, device=device)
            if g:
                self._guarded.append((whole, g, n))
            bufs.append(whole[g:g + n])
        self.slot_mem, self.workspace = bufs
        ptrs = (c_void_p * self.L)(*[c_void_p(b.data_ptr()) for b in self.banks])
        h = c_void_p()
        rc = lib().exmoe_cache_create(byref(h), byref(_shape(shape)), self.L, self.C, ptrs,
                                      c_void_p(self.slot_mem.data_ptr()), c_void_p(self.workspace.data_ptr()),
                                      self.max_tokens, int(wave_cap))
        _check(rc, "exmoe_cache_create")
        self.handle = h
        self.max_waves = -(-shape.num_experts // self.wave_cap)
        self.n_keys = self.max_waves * self.C

    # exmoe_moe_forward
    def forward(self, layer, hidden, topk_ids, topk_weights, out=None, stream=None):
        T = hidden.shape[0]
        if out is None:
            out = torch.empty_like(hidden)
        rc = lib().exmoe_moe_forward(self.handle, int(layer), _dev(hidden, torch.bfloat16, "hidden"),
                                     _dev(topk_ids, torch.int32, "topk_ids"), _dev(topk_weights, torch.float32, "topk_weights"),
                                     int(T), _dev(out, torch.bfloat16, "out"), _stream_ptr(stream))
        _check(rc, "exmoe_moe_forward")
        return out

    # exmoe_moe_forward_host
    def forward_host(self, layer, hidden, topk_ids, topk_weights, out=None, stream=None):
        """Host tensors in, host tensor out (synchronous): hidden BF16 [T, H], ids int32 [T, k], weights fp32 [T, k]."""
        T = int(hidden.shape[0])
        for t, dt, what in ((hidden, torch.bfloat16, "hidden"), (topk_ids, torch.int32, "topk_ids"),
                            (topk_weights, torch.float32, "topk_weights")):
            if t.is_cuda or t.dtype != dt or not t.is_contiguous():
                raise ValueError(f"{what}: need a contiguous CPU tensor of {dt}")
        if out is None:
            out = torch.empty((T, self.shape.d_model), dtype=torch.bfloat16)
        elif out.is_cuda or out.dtype != torch.bfloat16 or not out.is_contiguous():
            raise ValueError("out: need a contiguous CPU tensor of torch.bfloat16")
        rc = lib().exmoe_moe_forward_host(self.handle, int(layer), c_void_p(hidden.data_ptr()), c_void_p(topk_ids.data_ptr()),
                                          c_void_p(topk_weights.data_ptr()), T, c_void_p(out.data_ptr()), _stream_ptr(stream))
        _check(rc, "exmoe_moe_forward_host")
        return out

    def state(self, layer):
        E, C = self.shape.num_experts, self.C
        es = torch.empty(E, dtype=torch.int32)
        se = torch.empty(C, dtype=torch.int32)
        stamp = torch.empty(C, dtype=torch.int64)
        tick = torch.empty(1, dtype=torch.int64)
        _check(lib().exmoe_cache_get_state(self.handle, layer, es.data_ptr(), se.data_ptr(), stamp.data_ptr(),
                                           tick.data_ptr()), "exmoe_cache_get_state")
        return es.numpy(), se.numpy(), stamp.numpy().astype("uint64"), int(tick[0])

    def last_plan(self, layer, n_pairs):
        E = self.shape.num_experts
        hdr = [c_int32() for _ in range(3)]
        wave_of = torch.empty(E, dtype=torch.int32)
        slot_of = torch.empty(E, dtype=torch.int32)
        counts = torch.empty(self.n_keys, dtype=torch.int32)
        offsets = torch.empty(self.n_keys + 1, dtype=torch.int32)
        perm = torch.full((max(n_pairs, 1),), -1, dtype=torch.int32)
        misses = torch.empty(3 * E, dtype=torch.int32)
        rc = lib().exmoe_debug_last_plan(self.handle, layer, ctypes.addressof(hdr[0]), ctypes.addressof(hdr[1]),
                                         ctypes.addressof(hdr[2]), wave_of.data_ptr(), slot_of.data_ptr(),
                                         counts.data_ptr(), offsets.data_ptr(), perm.data_ptr(), misses.data_ptr())
        _check(rc, "exmoe_debug_last_plan")
        n_valid = int(offsets[-1])
        nm = hdr[2].value
        return {"n_active": hdr[0].value, "n_waves": hdr[1].value, "n_misses": nm,
                "wave_of": wave_of.numpy(), "slot_of": slot_of.numpy(), "counts": counts.numpy(),
                "offsets": offsets.numpy(), "perm": perm.numpy()[:n_valid],
                "misses": [tuple(int(x) for x in misses[3 * i:3 * i + 3]) for i in range(nm)]}

    def last_path(self):
        """PATH_* of the kernel family that served the most recent forward (exmoe_debug_last_path)."""
        rc = int(lib().exmoe_debug_last_path(self.handle))
        if rc < 0:
            raise ExmoeError(rc, "exmoe_debug_last_path")
        return rc

    def last_host_copy_bytes(self):
        n = c_size_t()
        _check(lib().exmoe_debug_last_host_copy_bytes(self.handle, byref(n)), "exmoe_debug_last_host_copy_bytes")
        return n.value

    def guards_intact(self):
        """True if every guard byte around slot memory and workspace still holds GUARD_BYTE (synchronises)."""
        torch.cuda.synchronize()
        for whole, g, n in self._guarded:
            if not bool((whole[:g] == self.GUARD_BYTE).all()) or not bool((whole[g + n:] == self.GUARD_BYTE).all()):
                return False
        return True

    def read_slot(self, layer, slot):
        out = torch.empty(self.bytes_per_expert, dtype=torch.uint8)
        _check(lib().exmoe_debug_read_slot(self.handle, layer, slot, out.data_ptr()), "exmoe_debug_read_slot")
        return out.numpy()

    def wait_timeout_selftest(self, budget_cycles=2_000_000):
        """Run the bounded-wait self-test kernel; returns the flag word (3 = gave up and raised the abort flag)."""
        v = c_int()
        _check(lib().exmoe_debug_wait_timeout(self.handle, int(budget_cycles), byref(v)), "exmoe_debug_wait_timeout")
        return v.value

    def stats(self, layer):
        s = exmoe_stats()
        _check(lib().exmoe_cache_stats(self.handle, layer, byref(s)), "exmoe_cache_stats")
        return {k: int(getattr(s, k)) for k, _ in exmoe_stats._fields_}

    # exmoe_cache_set_miss_path
    def set_miss_path(self, mode):
        """mode: MISS_DEVICE_FETCH (the default when the banks are mapped: no host wait, graph-capturable with C < E)
        or MISS_HOST_COPIES (plan read back once per call, one host-issued copy per miss on the copy stream)."""
        _check(lib().exmoe_cache_set_miss_path(self.handle, int(mode)), "exmoe_cache_set_miss_path")

    # exmoe_cache_prefetch
    def prefetch(self, layer, expert_ids, stream=None):
        _check(lib().exmoe_cache_prefetch(self.handle, int(layer), _dev(expert_ids, torch.int32, "expert_ids"),
                                          int(expert_ids.numel()), _stream_ptr(stream)), "exmoe_cache_prefetch")

    def reset(self, layer):
        _check(lib().exmoe_cache_reset(self.handle, layer), "exmoe_cache_reset")

    def status(self):
        return int(lib().exmoe_status(self.handle))

    def profile_enable(self, on=True, only=0):
        """on: bracket kernels with events; only: 0 all kernels, 1 gate/up, 2 down, 3 combine (timing runs)."""
        _check(lib().exmoe_profile_enable(self.handle, int(bool(on)) | (int(only) << 4)), "exmoe_profile_enable")

    def profile_read(self, kind):
        """(total event ms, bracketed launches) of kind 0 plan, 1 gate/up, 2 down, 3 combine, 4 miss copies."""
        ms, n = ctypes.c_double(), c_uint64()
        _check(lib().exmoe_profile_read(self.handle, int(kind), byref(ms), byref(n)), "exmoe_profile_read")
        return ms.value, int(n.value)

    def profile_overlap(self):
        """(ms of bracketed miss traffic, ms of it that ran while a bracketed GEMM kernel ran) since profile_enable."""
        a, b = ctypes.c_double(), ctypes.c_double()
        _check(lib().exmoe_profile_overlap(self.handle, byref(a), byref(b)), "exmoe_profile_overlap")
        return a.value, b.value

    def close(self):
        if getattr(self, "handle", None):
            lib().exmoe_cache_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
