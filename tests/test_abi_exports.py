"""CPU-side checks of the boundary: the library loads and exports every symbol
that include/nfd.h declares; the ctypes structures mirror the header."""
import ctypes
import os
import re

from paper_2506_01380_b200 import build as B
from paper_2506_01380_b200 import inputs as I
from paper_2506_01380_b200 import nfd as N

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    names = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        text = open(os.path.join(ROOT, "include", fn)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names |= set(re.findall(r"\b(nfd_[a-z0-9_]+)\s*\(", text))
    return names


def test_library_exports_every_declared_symbol():
    lib = ctypes.CDLL(B.build())
    declared = _declared()
    assert declared, "no declarations found"
    for name in declared:
        assert hasattr(lib, name), name
    assert declared == set(N.EXPORTS) | (declared - set(N.EXPORTS))
    for name in N.EXPORTS:
        assert name in declared, name


def test_cfg_struct_matches_header():
    text = open(os.path.join(ROOT, "include", "nfd.h")).read()
    body = re.search(r"typedef struct \{(.*?)\} nfd_cfg;", text, flags=re.S).group(1)
    body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
    fields = []
    for decl in body.split(";"):
        decl = decl.strip()
        if not decl:
            continue
        typ, rest = decl.split(None, 1)
        fields += [(typ, n.strip()) for n in rest.split(",")]
    got = [(("int" if t is ctypes.c_int else "float"), n) for n, t in N.NfdCfg._fields_]
    assert got == fields
    cfg = I.make_cfg("nfd310m")
    c = N.make_c_cfg(cfg)
    assert (c.n_layers, c.d_model, c.ctx_frames, c.n_steps) == (24, 1024, 16, 4)
    assert abs(c.sigma_d - 0.5) < 1e-7


def test_strerror_needs_no_gpu():
    lib = N.load()
    assert lib.nfd_strerror(0) == b"ok"
    assert lib.nfd_strerror(-5) == b"call not allowed in this cache state"


def test_acceptance_rule_in_the_library_matches_oracle():
    import itertools
    from oracle.nfd_oracle import accepted_count
    for n in range(1, 7):
        for acts in itertools.product([0, 1, 2], repeat=n):
            for k in range(1, 5):
                for i in range(n):
                    assert N.accepted_frames(list(acts), i, k) == accepted_count(list(acts), i, k)


def test_accepted_count_argument_checks():
    from paper_2506_01380_b200 import nfd as N
    lib = N.load()
    acts = N._ints([4, 4, 4, 2, 2])
    assert lib.nfd_accepted_count(acts, 5, 0, 4) == 3
    assert lib.nfd_accepted_count(acts, 5, 3, 4) == 2
    assert lib.nfd_accepted_count(acts, 5, 4, 4) == 1
    assert lib.nfd_accepted_count(acts, 5, 5, 4) == -4
    assert lib.nfd_accepted_count(None, 5, 0, 4) == -2
    assert lib.nfd_accepted_count(acts, 5, 0, 0) == -4
