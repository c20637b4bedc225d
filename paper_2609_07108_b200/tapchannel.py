"""Thin ctypes binding of the TapChannel library (`include/tap_channel.h`).

Paper Section 3.3: a per-source mailbox on the draft stage, written by the tap-producing
pipeline stages on a side path and read by the draft right before its own forward, with a
sequence stamp per slot.  Argument marshalling only; the handshake lives in the library.
"""
from __future__ import annotations

import ctypes as C
import os

from . import build as _build

OK, EINVAL, ESYS, ECUDA, ETIMEOUT, ESTATE = 0, -1, -2, -3, -4, -5
EXPORTS = ("tap_status_string", "tap_last_cuda_error", "tap_payload_bytes", "tap_ctrl_create", "tap_ctrl_attach",
           "tap_ctrl_close", "tap_ctrl_sources", "tap_ctrl_slot_bytes", "tap_ctrl_stamp", "tap_ctrl_publish",
           "tap_ctrl_reserve", "tap_ctrl_commit", "tap_ctrl_wait", "tap_ctrl_clear", "tap_mailbox_create",
           "tap_mailbox_ipc_handle", "tap_mailbox_slot", "tap_mailbox_slot_bytes", "tap_mailbox_wait",
           "tap_mailbox_release", "tap_mailbox_destroy", "tap_source_open", "tap_source_send", "tap_source_close")

_LIB = None


class TapError(RuntimeError):
    def __init__(self, code, what):
        self.code = code
        super().__init__(f"{what}: {lib().tap_status_string(code).decode()} (status {code}, "
                         f"cuda error {lib().tap_last_cuda_error()})")


def lib():
    global _LIB
    if _LIB is None:
        path = _build.TAP_LIB_PATH
        if not os.path.exists(path):
            raise ImportError(f"{path} is missing: build it with `python -m paper_2609_07108_b200.build`")
        l = C.CDLL(path)
        vp, u64, i = C.c_void_p, C.c_uint64, C.c_int
        sig = {
            "tap_status_string": (C.c_char_p, [i]),
            "tap_last_cuda_error": (i, []),
            "tap_payload_bytes": (u64, [u64, C.POINTER(C.c_uint32), i, C.c_uint32]),
            "tap_ctrl_create": (i, [C.c_char_p, i, u64, C.POINTER(vp)]),
            "tap_ctrl_attach": (i, [C.c_char_p, C.POINTER(vp)]),
            "tap_ctrl_close": (i, [vp, i]),
            "tap_ctrl_sources": (i, [vp]),
            "tap_ctrl_slot_bytes": (u64, [vp]),
            "tap_ctrl_stamp": (u64, [vp, i]),
            "tap_ctrl_publish": (i, [vp, i, u64, u64]),
            "tap_ctrl_reserve": (i, [vp, i, u64]),
            "tap_ctrl_commit": (i, [vp, i, u64, u64]),
            "tap_ctrl_wait": (i, [vp, i, u64, C.c_double, C.POINTER(u64)]),
            "tap_ctrl_clear": (i, [vp, i, u64]),
            "tap_mailbox_create": (i, [C.c_char_p, i, u64, C.POINTER(vp)]),
            "tap_mailbox_ipc_handle": (i, [vp, vp]),
            "tap_mailbox_slot": (vp, [vp, i]),
            "tap_mailbox_slot_bytes": (u64, [vp]),
            "tap_mailbox_wait": (i, [vp, i, u64, C.c_double, C.POINTER(u64)]),
            "tap_mailbox_release": (i, [vp, i, u64, vp]),
            "tap_mailbox_destroy": (i, [vp]),
            "tap_source_open": (i, [C.c_char_p, i, vp, vp, C.POINTER(vp)]),
            "tap_source_send": (i, [vp, vp, u64, u64, vp, C.c_double]),
            "tap_source_close": (i, [vp]),
        }
        for name, (res, args) in sig.items():
            f = getattr(l, name)
            f.restype, f.argtypes = res, args
        _LIB = l
    return _LIB


def _check(rc, what):
    if rc != 0:
        raise TapError(rc, what)


def payload_bytes(n_rows, feature_dims, elem_bytes=2):
    """Eq. (tap-comm): b * n * sum_s d_s."""
    arr = (C.c_uint32 * len(feature_dims))(*feature_dims)
    return int(lib().tap_payload_bytes(n_rows, arr, len(feature_dims), elem_bytes))


class Ctrl:
    """The stamps of a mailbox, in host shared memory (usable without a GPU)."""

    def __init__(self, name, n_sources=None, slot_bytes=None):
        self.h = C.c_void_p()
        self.owner = n_sources is not None
        if self.owner:
            _check(lib().tap_ctrl_create(name.encode(), n_sources, slot_bytes, C.byref(self.h)), "tap_ctrl_create")
        else:
            _check(lib().tap_ctrl_attach(name.encode(), C.byref(self.h)), "tap_ctrl_attach")

    def stamp(self, source):
        return int(lib().tap_ctrl_stamp(self.h, source))

    def publish(self, source, seq, nbytes):
        _check(lib().tap_ctrl_publish(self.h, source, seq, nbytes), "tap_ctrl_publish")

    def reserve(self, source, seq):
        _check(lib().tap_ctrl_reserve(self.h, source, seq), "tap_ctrl_reserve")

    def commit(self, source, seq, nbytes):
        _check(lib().tap_ctrl_commit(self.h, source, seq, nbytes), "tap_ctrl_commit")

    def wait(self, source, want, timeout_s):
        n = C.c_uint64()
        _check(lib().tap_ctrl_wait(self.h, source, want, timeout_s, C.byref(n)), "tap_ctrl_wait")
        return int(n.value)

    def clear(self, source, seq):
        _check(lib().tap_ctrl_clear(self.h, source, seq), "tap_ctrl_clear")

    def close(self):
        if self.h:
            lib().tap_ctrl_close(self.h, 1 if self.owner else 0)
            self.h = None


class Mailbox:
    """Draft side: n_sources device slots plus their stamps."""

    def __init__(self, name, n_sources, slot_bytes):
        self.h = C.c_void_p()
        _check(lib().tap_mailbox_create(name.encode(), n_sources, slot_bytes, C.byref(self.h)), "tap_mailbox_create")
        self.n_sources = n_sources
        self.slot_bytes = int(lib().tap_mailbox_slot_bytes(self.h))

    def ipc_handle(self) -> bytes:
        buf = C.create_string_buffer(64)
        _check(lib().tap_mailbox_ipc_handle(self.h, buf), "tap_mailbox_ipc_handle")
        return buf.raw

    def slot_ptr(self, source) -> int:
        return int(lib().tap_mailbox_slot(self.h, source))

    def slot_tensor(self, source, nbytes=None):
        """uint8 torch view of a slot (no copy)."""
        import torch
        n = self.slot_bytes if nbytes is None else nbytes

        class _Arr:
            __cuda_array_interface__ = {"shape": (n,), "typestr": "|u1", "data": (self.slot_ptr(source), False), "version": 2}

        return torch.as_tensor(_Arr(), device="cuda")

    def wait(self, source, seq, timeout_s):
        n = C.c_uint64()
        _check(lib().tap_mailbox_wait(self.h, source, seq, timeout_s, C.byref(n)), "tap_mailbox_wait")
        return int(n.value)

    def release(self, source, seq, stream_ptr):
        _check(lib().tap_mailbox_release(self.h, source, seq, C.c_void_p(stream_ptr)), "tap_mailbox_release")

    def destroy(self):
        if self.h:
            lib().tap_mailbox_destroy(self.h)
            self.h = None


class Source:
    """Source side: writes the taps of one pipeline stage into its slot of the mailbox."""

    def __init__(self, name, source, ipc_handle: bytes = None, local_slots: int = None):
        self.h = C.c_void_p()
        hbuf = C.create_string_buffer(ipc_handle, 64) if ipc_handle is not None else None
        _check(lib().tap_source_open(name.encode(), source, hbuf, C.c_void_p(local_slots or 0), C.byref(self.h)),
               "tap_source_open")

    def send(self, taps, seq, stream_ptr, timeout_s):
        """`taps`: a contiguous CUDA tensor; returns once the copy and the publication are queued."""
        if not taps.is_cuda or not taps.is_contiguous():
            raise ValueError("taps: a contiguous CUDA tensor is required")
        nbytes = taps.numel() * taps.element_size()
        _check(lib().tap_source_send(self.h, C.c_void_p(taps.data_ptr()), nbytes, seq, C.c_void_p(stream_ptr),
                                     timeout_s), "tap_source_send")

    def close(self):
        if self.h:
            lib().tap_source_close(self.h)
            self.h = None
