"""TapChannel host logic on CPU: the stamp handshake of the mailbox (control block in
host shared memory), its bounded waits, and a producer process that follows it."""
import ctypes
import os
import re
import subprocess
import sys
import textwrap
import time

import pytest

from paper_2609_07108_b200 import tapchannel as tap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_tap_library_exports_every_declared_symbol():
    from paper_2609_07108_b200 import build
    lib = ctypes.CDLL(build.build_tap())
    header = open(os.path.join(ROOT, "include", "tap_channel.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    header = re.sub(r"^\s*#.*$", "", header, flags=re.M)
    names = re.findall(r"\b([A-Za-z_][A-Za-z0-9_]*)\s*\([^;{]*\)\s*;", header)
    assert len(names) >= 20
    for name in names:
        assert hasattr(lib, name), f"{name} declared in the header but not exported"
    assert set(tap.EXPORTS) == set(names)


def test_payload_volume_is_eq_tap_comm():
    # b * n * sum_s d_s: 4096 token rows, embedding width 4096 from the first stage, hidden 4096 from two more
    assert tap.payload_bytes(4096, [4096, 4096, 4096], 2) == 2 * 4096 * 3 * 4096
    assert tap.payload_bytes(10, [], 2) == 0


def test_stamp_handshake_and_its_violations():
    name = f"/tap_test_{os.getpid()}_a"
    c = tap.Ctrl(name, n_sources=3, slot_bytes=1024)
    try:
        assert [c.stamp(s) for s in range(3)] == [0, 0, 0]
        c.publish(1, 7, 512)
        assert c.stamp(1) == 7 and c.wait(1, 7, 0.1) == 512
        with pytest.raises(tap.TapError) as e:           # the slot is full: a second write must wait for the reader
            c.publish(1, 8, 100)
        assert e.value.code == tap.ESTATE
        with pytest.raises(tap.TapError) as e:           # the reader hands back the sequence it read, nothing else
            c.clear(1, 6)
        assert e.value.code == tap.ESTATE
        c.clear(1, 7)
        assert c.stamp(1) == 0
        # asynchronous writer: reserved taps are not readable, and nobody else can take the slot
        c.reserve(2, 9)
        assert c.stamp(2) not in (0, 9)
        with pytest.raises(tap.TapError) as e:
            c.wait(2, 9, 0.05)
        assert e.value.code == tap.ETIMEOUT
        with pytest.raises(tap.TapError) as e:
            c.reserve(2, 10)
        assert e.value.code == tap.ESTATE
        c.commit(2, 9, 64)
        assert c.wait(2, 9, 0.05) == 64
        for bad in (lambda: c.publish(5, 1, 1), lambda: c.publish(0, 0, 1), lambda: c.publish(0, 1, 4096)):
            with pytest.raises(tap.TapError) as e:
                bad()
            assert e.value.code == tap.EINVAL
        # a second mapping of the same block sees the same stamps
        d = tap.Ctrl(name)
        assert d.stamp(2) == 9
        d.clear(2, 9)
        assert c.stamp(2) == 0
        d.close()
    finally:
        c.close()
    with pytest.raises(tap.TapError) as e:               # the name is gone with its creator
        tap.Ctrl(name)
    assert e.value.code == tap.ESYS


def test_wait_is_bounded():
    c = tap.Ctrl(f"/tap_test_{os.getpid()}_b", n_sources=1, slot_bytes=64)
    try:
        t0 = time.perf_counter()
        with pytest.raises(tap.TapError) as e:
            c.wait(0, 1, 0.2)                            # nobody ever writes
        dt = time.perf_counter() - t0
        assert e.value.code == tap.ETIMEOUT and 0.15 < dt < 2.0
    finally:
        c.close()


def test_producer_process_follows_the_handshake():
    """Three sources in another process write five microbatches each; the reader takes them in
    microbatch order.  A writer can never overwrite taps that have not been read: it waits for
    the stamp to return to 0."""
    name = f"/tap_test_{os.getpid()}_c"
    n_sources, n_micro = 3, 5
    c = tap.Ctrl(name, n_sources=n_sources, slot_bytes=1 << 20)
    try:
        child = subprocess.Popen([sys.executable, "-c", textwrap.dedent(f"""
            import sys, time, random
            sys.path.insert(0, {ROOT!r})
            from paper_2609_07108_b200 import tapchannel as tap
            c = tap.Ctrl({name!r})
            random.seed(1)
            for m in range(1, {n_micro} + 1):
                for s in range({n_sources}):
                    c.wait(s, 0, 20.0)                    # slot handed back by the reader
                    time.sleep(random.random() * 0.01)
                    c.publish(s, m, 1000 * m + s)         # the size field carries a recognisable value
            c.close()
            print("WRITER DONE")
        """)], stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True)
        got = []
        for m in range(1, n_micro + 1):
            for s in range(n_sources):
                got.append(c.wait(s, m, 20.0))
                time.sleep(0.002)                         # "reading" the slot
                assert c.stamp(s) == m                    # still mine: the writer is held off
                c.clear(s, m)
        out, err = child.communicate(timeout=60)
        assert child.returncode == 0, err[-2000:]
        assert "WRITER DONE" in out
        assert got == [1000 * m + s for m in range(1, n_micro + 1) for s in range(n_sources)]
    finally:
        c.close()
