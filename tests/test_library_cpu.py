"""Host-side checks of the CUDA library that need no GPU: it builds, loads, exports every symbol
the header declares, and its loader validates blobs before touching the device."""
import ctypes
import os
import re
import struct

import numpy as np
import pytest

from workloads import complete_catalog, crossbar_catalog, crossbar_topology, node_template_catalog, tree_topology

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2609_34340_b200.build import build
    return ctypes.CDLL(build())


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(ROOT, "include", "variopath.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    names = sorted(set(re.findall(r"\b(vp_[a-z_]+)\s*\(", header)))
    assert len(names) >= 13
    for n in names:
        assert hasattr(lib, n), f"{n} declared in variopath.h but not exported"


def test_strerror(lib):
    lib.vp_strerror.restype = ctypes.c_char_p
    assert lib.vp_strerror(0) == b"ok"
    assert b"catalog" in lib.vp_strerror(-2)
    assert b"unknown" in lib.vp_strerror(-99)


def _load(lib, topo, chan):
    h = ctypes.c_void_p()
    lib.vp_load_catalog.argtypes = [ctypes.c_char_p, ctypes.c_size_t, ctypes.c_char_p, ctypes.c_size_t,
                                    ctypes.c_int, ctypes.POINTER(ctypes.c_void_p)]
    rc = lib.vp_load_catalog(topo, len(topo), chan, len(chan), 0, ctypes.byref(h))
    if rc == 0:
        lib.vp_free_catalog.argtypes = [ctypes.c_void_p]
        lib.vp_free_catalog(h)
    return rc


def test_loader_validates_before_using_the_device(lib):
    cat = complete_catalog(tree_topology(1))
    topo, chan = cat.topology.blob(), cat.blob()
    ok = _load(lib, topo, chan)
    assert ok in (0, -4)                     # -4 (no CUDA device) only on a CPU-only box
    n_shapes, n_fam, nnz = struct.unpack_from("<3I", chan, 12)
    nnz_off = 24 + 4 * (n_shapes + 1)
    fam_off = nnz_off + 8 * nnz + 4 * (n_shapes + 1)
    assert _load(lib, topo, chan[:-2]) == -2                      # truncated
    assert _load(lib, topo[:40], chan) == -2
    assert _load(lib, b"XXXX" + topo[4:], chan) == -2             # bad magic
    bad = bytearray(chan)                                         # Eq. (3): unbalanced shape
    struct.pack_into("<H", bad, nnz_off + 4, struct.unpack_from("<H", bad, nnz_off + 4)[0] + 1)
    assert _load(lib, topo, bytes(bad)) == -2
    fams = np.frombuffer(chan, dtype="<u2", offset=fam_off).reshape(n_fam, 8).copy()
    inst = cat.topology.instances                                 # Eq. (4): one PXB path used by two lanes
    pxb = next(i for i, r in enumerate(inst) if r.kind == 1 and r.src_group == 0)
    nic = next(i for i, r in enumerate(inst) if r.kind == 2 and r.src_group == 0)
    f = next(i for i in range(n_fam) if pxb in fams[i] and nic in fams[i])
    fams[f][list(fams[f]).index(nic)] = pxb
    fams[f].sort()
    bad = bytearray(chan)
    bad[fam_off:] = fams.astype("<u2").tobytes()
    assert _load(lib, topo, bytes(bad)) == -2
    bad = bytearray(chan)                                         # family that does not realise its shape
    fams = np.frombuffer(chan, dtype="<u2", offset=fam_off).reshape(n_fam, 8).copy()
    fams[0], fams[-1] = fams[-1].copy(), fams[0].copy()
    bad[fam_off:] = fams.astype("<u2").tobytes()
    assert _load(lib, topo, bytes(bad)) == -2
    big = crossbar_catalog(crossbar_topology(6))                  # group size 6 > 4
    assert _load(lib, big.topology.blob(), big.blob()) == -6
    assert lib.vp_load_catalog(None, 0, None, 0, 0, None) == -1


def test_bad_arguments_without_a_device(lib):
    lib.vp_pack_workspace_bytes.restype = ctypes.c_size_t
    assert lib.vp_pack_workspace_bytes(16, 1024, 8, 128) % 256 == 0
    assert lib.vp_pack_workspace_bytes(16, 1024, 8, 128) > 1024 * 8 * 4
    assert lib.vp_pack_workspace_bytes(0, 1024, 8, 128) == 0
    lib.vp_kernel_launch_count.restype = ctypes.c_int64
    assert lib.vp_kernel_launch_count() == 0
    null = ctypes.c_void_p()
    assert lib.vp_pack(null, null, null, null, 16, 0, 8, null, 4, 2, 1, null, ctypes.c_int64(16), null,
                       ctypes.c_int64(0), null, null, null, ctypes.c_size_t(0), null) == -1


def test_binding_fails_loudly_without_library(monkeypatch):
    import paper_2609_34340_b200.binding as b
    monkeypatch.setattr(b, "_lib", None)
    monkeypatch.setattr(b, "_LIB_PATH", "/nonexistent/libvariopath.so")
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        b.kernel_launch_count()


def test_status_bits_are_distinct_and_the_timeout_bit_is_declared():
    """Every status bit the header declares is mirrored by the binding, no two share a value, and the row-copy
    kernels' give-up bit (the output buffer is incomplete) is among them."""
    import paper_2609_34340_b200 as vp
    header = open(os.path.join(ROOT, "include", "variopath.h")).read()
    declared = dict(re.findall(r"#define (VP_ST_[A-Z_]+)\s+\(?([0-9 <]+)\)?", header))
    values = {k: eval(v) for k, v in declared.items()}
    assert len(set(values.values())) == len(values) and "VP_ST_INTERNAL_TIMEOUT" in values
    for name, v in values.items():
        assert getattr(vp, name[3:]) == v, name
    assert vp.ST_INTERNAL_TIMEOUT == 1 << 30 and vp.ST_INTERNAL_TIMEOUT & (vp.ST_PACK_MISMATCH | vp.ST_PACK_CAPACITY) == 0
