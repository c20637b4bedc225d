"""TapChannel on a GPU: the taps of several source stages cross from another process into
the draft process's mailbox through CUDA IPC, ordered by the slots' sequence stamps.
All waiting is on the host and bounded; no kernel of one process waits for the other."""
import os
import subprocess
import sys
import textwrap
import time

import pytest
import torch

from paper_2609_07108_b200 import tapchannel as tap

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

N_ROWS = 4096                      # token rows of a microbatch
DIMS = [2048, 4096, 4096]          # per-source feature width (first stage: embedding width)
N_MICRO = 6


def pattern(source, micro):
    return float(source + 1) + micro / 16.0          # exact in bf16


def test_taps_cross_processes_through_the_mailbox(tmp_path):
    assert torch.cuda.is_available()
    name = f"/tap_gpu_{os.getpid()}"
    slot_bytes = N_ROWS * max(DIMS) * 2
    mb = tap.Mailbox(name, len(DIMS), slot_bytes)
    try:
        (tmp_path / "handle.hex").write_text(mb.ipc_handle().hex())
        child = subprocess.Popen([sys.executable, "-c", textwrap.dedent(f"""
            import sys
            sys.path.insert(0, {ROOT!r})
            import torch
            from paper_2609_07108_b200 import tapchannel as tap
            handle = bytes.fromhex(open({str(tmp_path / 'handle.hex')!r}).read())
            dims = {DIMS!r}
            srcs = [tap.Source({name!r}, s, ipc_handle=handle) for s in range(len(dims))]
            stream = torch.cuda.current_stream().cuda_stream
            taps = {{(m, s): torch.full(({N_ROWS}, d), float(s + 1) + m / 16.0, dtype=torch.bfloat16, device="cuda")
                    for m in range(1, {N_MICRO} + 1) for s, d in enumerate(dims)}}
            torch.cuda.synchronize()
            for m in range(1, {N_MICRO} + 1):
                for s, d in enumerate(dims):
                    srcs[s].send(taps[(m, s)], m, stream, 60.0)   # waits (bounded) until the draft has read microbatch m - 1
            torch.cuda.synchronize()
            for x in srcs:
                x.close()
            print("SOURCES DONE")
        """)], stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True)
        stream = torch.cuda.current_stream().cuda_stream
        total, t0 = 0, None
        for m in range(1, N_MICRO + 1):
            for s, d in enumerate(DIMS):
                nbytes = mb.wait(s, m, 120.0)
                t0 = t0 or time.perf_counter()
                assert nbytes == N_ROWS * d * 2
                view = mb.slot_tensor(s, nbytes).view(torch.bfloat16)
                bad = torch.count_nonzero(view != pattern(s, m))       # the draft's read of the slot, on its stream
                mb.release(s, m, stream)                             # handed back once that read has run
                assert int(bad.item()) == 0, (s, m)
                total += nbytes
        dt = time.perf_counter() - t0
        out, err = child.communicate(timeout=120)
        assert child.returncode == 0, err[-3000:]
        assert "SOURCES DONE" in out
        assert total == N_MICRO * tap.payload_bytes(N_ROWS, DIMS, 2)   # Eq. tap-comm, every feature crossed once
        print(f"[tap] {total / 1e6:.0f} MB in {dt * 1e3:.1f} ms through CUDA IPC, stamps in host shared memory "
              f"({total / dt / 1e9:.1f} GB/s incl. the handshake)")
        # all slots are empty again
        torch.cuda.synchronize()
        ctrl = tap.Ctrl(name)                                        # a second mapping of the stamps
        assert [ctrl.stamp(s) for s in range(len(DIMS))] == [0] * len(DIMS)
        ctrl.close()
    finally:
        mb.destroy()


def test_same_process_source_and_bounded_waits():
    name = f"/tap_gpu_{os.getpid()}_b"
    mb = tap.Mailbox(name, 2, 1 << 20)
    try:
        with pytest.raises(tap.TapError) as e:       # nothing was sent: the draft's wait runs out
            mb.wait(0, 1, 0.2)
        assert e.value.code == tap.ETIMEOUT
        src = tap.Source(name, 1, local_slots=mb.slot_ptr(0))
        side = torch.cuda.Stream()
        taps = torch.arange(1 << 18, dtype=torch.int32, device="cuda")
        with torch.cuda.stream(side):
            src.send(taps, 1, side.cuda_stream, 5.0)
            with pytest.raises(tap.TapError) as e:   # the slot is taken until the draft hands it back
                src.send(taps, 2, side.cuda_stream, 0.2)
            assert e.value.code == tap.ETIMEOUT
        assert mb.wait(1, 1, 10.0) == taps.numel() * 4
        got = mb.slot_tensor(1, taps.numel() * 4).view(torch.int32)
        assert torch.equal(got, taps)
        with pytest.raises(tap.TapError) as e:       # only the sequence that is there can be released
            mb.release(1, 3, torch.cuda.current_stream().cuda_stream)
        assert e.value.code == tap.ESTATE
        mb.release(1, 1, torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()
        with torch.cuda.stream(side):
            src.send(taps + 1, 2, side.cuda_stream, 5.0)      # the slot is free again
        assert mb.wait(1, 2, 10.0) == taps.numel() * 4
        assert torch.equal(mb.slot_tensor(1, taps.numel() * 4).view(torch.int32), taps + 1)
        mb.release(1, 2, torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()
        src.close()
    finally:
        mb.destroy()
