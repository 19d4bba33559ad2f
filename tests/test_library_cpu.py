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
    rc = lib.vp_load_catalog(topo, len(topo), chan, len(chan), -1, ctypes.byref(h))     # host-only handle: no GPU needed
    if rc == 0:
        lib.vp_free_catalog.argtypes = [ctypes.c_void_p]
        lib.vp_free_catalog(h)
    return rc


def test_loader_validates_before_using_the_device(lib):
    cat = complete_catalog(tree_topology(1))
    topo, chan = cat.topology.blob(), cat.blob()
    assert _load(lib, topo, chan) == 0
    for other in (complete_catalog(tree_topology(2, pcie_bw=64, nic_bw=50)), node_template_catalog(tree_topology(9, nic_bw=50)),
                  complete_catalog(tree_topology(1, g=3)), crossbar_catalog(crossbar_topology(4))):
        assert _load(lib, other.topology.blob(), other.blob()) == 0
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


def test_host_only_handle_info_and_refusals():
    """device = -1: the loader parses, validates and analyses without a GPU; calls that would launch refuse."""
    import paper_2609_34340_b200 as vp
    cat = complete_catalog(tree_topology(1))
    dc = vp.load_catalog(cat.topology.blob(), cat.blob(), device=-1)
    assert (dc.N, dc.G, dc.g, dc.n_shapes, dc.n_families, dc.covered, dc.node_symmetric) == (8, 2, 4, 3, 6, 1, 0)
    assert dc.row_patterns == 0 and dc.argmax_classes == 0 and len(vp.catalog_argmax_classes(dc)) == 0
    assert vp.schedule_workspace_bytes(dc, 4, vp.SchedParams()) == 0          # nothing can be launched from it
    with pytest.raises(vp.VpError) as e:
        vp.load_catalog(cat.topology.blob(), cat.blob()[:-2], device=-1)
    assert e.value.code == vp.E_BAD_CATALOG
    big = crossbar_catalog(crossbar_topology(6))
    with pytest.raises(vp.VpError) as e:
        vp.load_catalog(big.topology.blob(), big.blob(), device=-1)
    assert e.value.code == vp.E_UNSUPPORTED
    with pytest.raises(vp.VpError) as e:
        vp.load_catalog(cat.topology.blob(), cat.blob(), device=-2)
    assert e.value.code == vp.E_BAD_ARG
    uncovered = type(cat)(cat.topology, [cat.shapes[-1]], [cat.buckets[-1]])   # the all-PIX shape only
    assert vp.load_catalog(uncovered.topology.blob(), uncovered.blob(), device=-1).covered == 0


@pytest.mark.parametrize("nodes,nic_bw", [(2, 64), (5, 50), (16, 64), (32, 64)])
def test_argmax_classes_reproduce_every_shape(nodes, nic_bw):
    """The loader's class decomposition of Eq. (6)'s arg-max, checked against the catalog itself: every shape of a
    two-rail node-template catalog is (first row p0, second row p1); the decomposition claims that the shape of
    (p0, the second row at place j of the list of p0's class) is run_start(p0) + j.  Rebuilt here from the shapes'
    (a, d, count) lists alone: every claimed pair is that shape, and the claims cover every shape exactly once."""
    import paper_2609_34340_b200 as vp
    cat = node_template_catalog(tree_topology(nodes, pcie_bw=64, nic_bw=nic_bw))
    S = cat.topology.groups_per_node
    assert S == 2
    dc = vp.load_catalog(cat.topology.blob(), cat.blob(), device=-1)
    assert dc.node_symmetric == 1 and dc.argmax_classes > 0

    def row(shape, q):                      # terms leaving rail q of node 0: (table index of (delta, q, q'), lanes), by destination
        return tuple((((d // S) * S + q) * S + d % S, c) for (a, d, c) in shape if a == q)

    rows_of_shape = [(row(s, 0), row(s, 1)) for s in cat.shapes]
    assert dc.row_patterns == len({r for pair in rows_of_shape for r in pair})
    d = vp.catalog_argmax_classes(dc)
    n_chunks, stride, ent_off = int(d[0]), int(d[1]), int(d[2])
    n = dc.argmax_classes
    first = [int(x) for x in d[3:3 + 2 * n + 1]]
    assert first[0] == 0 and first[-1] == n_chunks and first == sorted(first)
    unit_of_chunk = [int(x) for x in d[3 + 2 * n + 1:3 + 2 * n + 1 + n_chunks]]
    assert unit_of_chunk == [u for u in range(2 * n) for _ in range(first[u + 1] - first[u])]

    def entries(unit):
        out = []
        for e in range(first[unit] * 32, first[unit + 1] * 32):
            words = d[ent_off + e * stride: ent_off + (e + 1) * stride]
            if int(words[-1]) == 0xFFFFFFFF:                     # padding comes last and scores nothing
                assert not any(int(w) for w in words[:-1])
                continue
            assert len(out) == e - first[unit] * 32              # no padding in between
            terms = tuple((int(w) & 0xFFFF, int(w) >> 16) for w in words[:-1] if int(w) >> 16)
            out.append((terms, int(words[-1])))
        return out

    seen = np.zeros(cat.n_shapes, dtype=np.int64)
    for cl in range(n):
        members, second = entries(2 * cl), entries(2 * cl + 1)
        assert members and second
        assert [t for _, t in second] == list(range(len(second)))               # places count up
        assert [t for _, t in members] == sorted({t for _, t in members})       # run starts in shape order
        for p0, run_start in members:
            for p1, place in second:
                assert rows_of_shape[run_start + place] == (p0, p1), (cl, run_start, place)
                seen[run_start + place] += 1
    assert (seen == 1).all()
