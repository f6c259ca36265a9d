"""Host-side checks of the C ABI that need no GPU: the library loads, exports every symbol the
header declares, validates its arguments, and lays out the hierarchy as the paper defines it."""
import ctypes
import os
import re

import pytest

import paper_2609_31093_b200 as P
from paper_2609_31093_b200 import binding as PB
from oracle import pisa_oracle as O

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_functions():
    names = []
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if not fn.endswith(".h"):
            continue
        src = open(os.path.join(ROOT, "include", fn)).read()
        src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
        names += re.findall(r"\b(pisa_[a-z_0-9]+)\s*\(", src)
    return sorted(set(names))


def test_library_exports_every_declared_symbol():
    lib = P.lib()
    decl = _declared_functions()
    assert len(decl) >= 12
    for name in decl:
        assert hasattr(lib, name), name
    assert lib.pisa_version() == 100


@pytest.mark.parametrize("N,C,g", [(1024, 64, 2), (32768, 64, 4), (131072, 128, 2), (1000, 24, 3), (50, 64, 2),
                                   (524288, 64, 2)])
def test_pyramid_layout_matches_paper_hierarchy(N, C, g):
    p = P.Params(1, N, 4, 2, 64, C, g, 8)
    L, M, off, nbytes = P.pyramid_layout(p)
    assert M == O.hierarchy(N, C, g) and L == len(M) - 1
    es = 2
    for l in range(1, L):
        assert off[l + 1] * es >= off[l] * es + 2 * M[l] * 64 * es      # levels do not overlap
        assert (off[l] * es) % 256 == 0
    assert nbytes >= off[L] * es + 2 * M[L] * 64 * es


def test_argument_validation():
    ok = P.Params(1, 1024, 4, 2, 64, 64, 2, 8)
    assert P.workspace_bytes(ok, PB.OP_FORWARD) >= 256
    bad = [
        dict(Hq=3),            # Hq % Hkv != 0
        dict(K=2),             # K < 3 (three forced blocks)
        dict(g=1),
        dict(N=0),
    ]
    for kw in bad:
        args = dict(B=1, N=1024, Hq=4, Hkv=2, d=64, C=64, g=2, K=8)
        args.update(kw)
        with pytest.raises(P.PisaError, match="invalid argument"):
            P.workspace_bytes(P.Params(**args), PB.OP_FORWARD)
    for kw in [dict(d=48), dict(K=64), dict(g=8, K=32), dict(Hq=6, Hkv=2)]:
        args = dict(B=1, N=1024, Hq=4, Hkv=2, d=64, C=64, g=2, K=8)
        args.update(kw)
        with pytest.raises(P.PisaError, match="unsupported"):
            P.workspace_bytes(P.Params(**args), PB.OP_FORWARD)
    nc = P.Params(1, 1024, 4, 2, 64, 64, 2, 8)
    nc.c.causal = 0
    with pytest.raises(P.PisaError, match="unsupported"):
        P.workspace_bytes(nc, PB.OP_FORWARD)
    # null pointers are rejected before anything is launched (no GPU needed to see that)
    lib = P.lib()
    assert lib.pisa_build_pyramid(ok.ref(), None, None, None) == -1
    assert lib.pisa_route(ok.ref(), None, None, None, None, None, None, None, 0, None) == -1
    assert lib.pisa_bsa_fwd(ok.ref(), None, None, None, None, None, None, None, None, 0, None) == -1
    assert lib.pisa_debug_wait_timeout(None, 1000, None) == -1
    assert lib.pisa_forward(ok.ref(), None, None, None, None, None, None, None, None, 0, None) == -1
    assert lib.pisa_status_string(-3).decode() == "workspace too small"


def test_host_arena_size_covers_its_slots():
    """The host entry point walks the KV heads with four slots of per-head tensors and two per-head
    workspaces and pyramids (two heads' kernels in flight, one head uploading, one downloading)."""
    p = P.Params(1, 8192, 16, 4, 128, 64, 2, 16)
    es, G = 2, 4
    unit = P.Params(1, 8192, G, 1, 128, 64, 2, 16)
    slot = 2 * 8192 * G * 128 * es + 2 * 8192 * 128 * es + G * 8192 * 4 + 8192 * 16 * 4
    need = 4 * slot + 2 * P.pyramid_layout(unit)[3] + 2 * P.workspace_bytes(unit, PB.OP_FORWARD)
    assert P.workspace_bytes(p, PB.OP_FORWARD_HOST) >= need


def test_packed_arena_sizes_cover_their_padded_tensors():
    """The packed entry points run a group of short sequences as a padded batch of at most 32768 tokens held in the
    workspace: the forward needs padded q, out, k, v, lse and idx beside a forward workspace and a pyramid, the
    backward padded q, out, dout, dq, k, v, dk, dv, lse and idx beside a backward workspace.  The backward's arena
    is refused (unsupported) where the backward itself is: fp32 inputs."""
    p = P.Params(1, 4096, 8, 2, 128, 64, 2, 4)
    es, tok = 2, 32768
    qb, kb = tok * 8 * 128 * es, tok * 2 * 128 * es
    lb, ib = tok * 8 * 4, tok * 2 * 4 * 4
    fwd = P.workspace_bytes(p, PB.OP_FORWARD_PACKED)
    assert fwd >= P.workspace_bytes(p, PB.OP_FORWARD) + 2 * qb + 2 * kb + lb + ib
    bwd = P.workspace_bytes(p, PB.OP_BSA_BWD_PACKED)
    assert bwd >= P.workspace_bytes(p, PB.OP_BSA_BWD) + 4 * qb + 4 * kb + lb + ib
    with pytest.raises(P.PisaError):
        P.workspace_bytes(P.Params(1, 4096, 8, 2, 32, 64, 2, 4, dtype="fp32"), PB.OP_BSA_BWD_PACKED)
