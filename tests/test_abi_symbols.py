"""The C-ABI library loads without a GPU and exports every function the headers under include/ declare."""
import glob
import os
import re

from conftest import ROOT


def declared_functions():
    text = "".join(open(h).read() for h in sorted(glob.glob(os.path.join(ROOT, "include", "*.h"))))
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(lc_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    from paper_2009_13003_b200 import binding

    names = declared_functions()
    assert "lc_compress" in names and "lc_recover" in names and len(names) >= 10
    L = binding.lib()
    for name in names:
        assert hasattr(L, name), name
    assert sorted(binding.SYMBOLS) == names


def test_host_side_size_functions_match_the_format_text(oracle):
    from paper_2009_13003_b200 import binding

    for n in (0, 1, 10, 4096, 4097, 61_706, 11_689_512, 1_315_575_808):
        for nbits in (1, 2, 5, 8, 9):
            nchunks = (n + 4095) // 4096
            head = (64 + 16 * 2 ** nbits + 8 * (nchunks + 1) + 64 * nchunks + 15) // 16 * 16
            want = head + (n * nbits + 7) // 8 + 16 * nchunks
            assert binding.stream_bound(n, nbits) == want == oracle.stream_bound(n, nbits)
        assert n <= binding.workspace_bytes(n) <= 1.01 * n + 131072
    assert binding.stream_bound(10, 0) == 0 and binding.stream_bound(10, 10) == 0


def test_host_argument_checks_need_no_device():
    from paper_2009_13003_b200 import binding

    L = binding.lib()
    assert L.lc_compress(None, None, 16, 4, None, 0, None, 0, None) == binding.ERR_ARG
    assert L.lc_recover(None, None, None, 0, 16, None, None, 0, None) == binding.ERR_ARG
    # lc_compress_update: the tracked state must be given, aligned, and must not be cur (made-up addresses:
    # the checks come before anything is touched)
    base, cur, stream, ws = 0x10000, 0x20000, 0x30000, 0x40000
    upd = lambda out, nbits=4: L.lc_compress_update(base, cur, 16, nbits, stream, 1 << 20, out, ws, 1 << 20, None)
    assert upd(None) == binding.ERR_ARG
    assert upd(cur) == binding.ERR_ARG
    assert upd(0x50004) == binding.ERR_ARG
    assert upd(0x50000, nbits=10) == binding.ERR_ARG
    assert L.lc_compress_update(base, cur, 16, 4, stream, 8, 0x50000, ws, 1 << 20, None) == binding.ERR_CAPACITY
    assert L.lc_strerror(binding.ERR_FORMAT) == b"malformed stream"
    # lc_compress_opt: unknown option bits are refused before anything else happens
    assert L.lc_compress_opt(base, cur, 16, 4, stream, 1 << 20, None, ws, 1 << 20, 8, None) == binding.ERR_ARG
    assert L.lc_compress_opt(base, cur, 16, 4, stream, 1 << 20, cur, ws, 1 << 20, 1, None) == binding.ERR_ARG


def test_launch_parameter_caches_are_per_device():
    # Function attributes and occupancy belong to a device: a function-scope static that caches them must be an
    # array indexed by the device ordinal (a process may use several GPUs).
    csrc = os.path.join(ROOT, "paper_2009_13003_b200", "csrc")
    for path in sorted(glob.glob(os.path.join(csrc, "*.cu"))):
        text = re.sub(r"//.*", "", open(path).read())
        for m in re.finditer(r"^\s+static\s+(?!_|const|constexpr)[^;(]*;", text, flags=re.M):
            decl = m.group(0)
            assert "[kMaxDevices]" in decl, "%s: %s" % (os.path.basename(path), decl.strip())
