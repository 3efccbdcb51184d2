"""CPU-side checks of the C-ABI library: it builds, loads, exports every declared symbol, and
rejects bad arguments on the host before touching a device.  No kernel is launched here."""
import ctypes as C
import os
import re

import pytest

from paper_2602_16994_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load_library()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "specverify.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\bint(?:32|64)_t\s+(spec_\w+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert set(names) == set(binding.EXPORTS)
    for n in names:
        assert getattr(lib, n) is not None


def test_struct_layout_matches_header():
    text = open(os.path.join(ROOT, "include", "specverify.h")).read()
    def fields(name):
        blocks = {nm: body for body, nm in re.findall(r"typedef struct \{(.*?)\} (\w+);", text, flags=re.S)}
        body = blocks[name]
        body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
        out = []
        for decl in body.split(";"):
            decl = decl.strip()
            if not decl:
                continue
            for nm in re.findall(r"[\*\s,](\w+)(?=\s*(?:,|$))", " " + decl):
                out.append(nm)
        return out
    assert fields("SpecIn") == [f[0] for f in binding.SpecIn._fields_]
    assert fields("SpecOut") == [f[0] for f in binding.SpecOut._fields_]


def good_in(**kw):
    d = dict(B=2, N=3, V=100, logits_dtype=1, target_logits=0x1000, draft_logits=0x1000, seq_stride=300,
             node_stride=100, parent=0x1000, topo_seq_stride=0, token=0x1000, temperature=1.0, top_k=0,
             top_p=1.0, temperature_per_seq=None, u_accept=0x1000, u_bonus=0x1000)
    d.update(kw)
    return binding.SpecIn(**d)


def good_out():
    return binding.SpecOut(accepted_node=0x1000, accept_len=0x1000, out_tokens=0x1000, bonus_token=0x1000,
                           status=0x1000)


def test_workspace_bytes(lib):
    n = C.c_int64()
    assert lib.spec_workspace_bytes(C.byref(good_in()), C.byref(n)) == 0 and n.value >= 2 * 3 * 8
    assert lib.spec_workspace_bytes(None, C.byref(n)) == -1
    assert lib.spec_workspace_bytes(C.byref(good_in(N=0)), C.byref(n)) == -2
    assert lib.spec_workspace_bytes(C.byref(good_in(N=5000)), C.byref(n)) == -2


@pytest.mark.parametrize("fn", ["spec_verify_specinfer", "spec_verify_traversal"])
def test_verify_rejects_bad_arguments_on_the_host(lib, fn):
    f = getattr(lib, fn)
    ws, nb = C.c_void_p(0x10000), 1 << 20
    call = lambda i, o=good_out(), w=ws, n=nb: f(C.byref(i), C.byref(o), w, n, None)
    assert f(None, C.byref(good_out()), ws, nb, None) == -1
    assert call(good_in(target_logits=None)) == -1
    assert call(good_in(u_bonus=None)) == -1
    assert call(good_in(), o=binding.SpecOut()) == -1
    assert call(good_in(B=0)) == -2
    assert call(good_in(node_stride=50)) == -2
    assert call(good_in(logits_dtype=2)) == -3
    assert call(good_in(temperature=0.0)) == -4
    assert call(good_in(temperature=float("nan"))) == -4
    assert call(good_in(top_p=0.0)) == -4
    assert call(good_in(top_p=1.5)) == -4
    assert call(good_in(top_k=-1)) == -4
    assert call(good_in(), w=None) == -5
    assert call(good_in(), w=C.c_void_p(0x10008)) == -5          # misaligned
    assert call(good_in(), n=16) == -5                           # too small
    assert call(good_in(V=1 << 30, node_stride=1 << 30)) == -6   # beyond the on-chip plan


def test_other_entry_points_reject_bad_arguments(lib):
    assert lib.spec_sample_bonus(None, 1, 10, None, None, None, None, 0, None) == -1
    assert lib.spec_sample_bonus(C.c_void_p(16), 0, 10, C.c_void_p(16), C.c_void_p(16), None, None, 0, None) == -2
    assert lib.spec_tree_probs(C.byref(good_in()), 2, C.c_void_p(16), None, None, 0, None) == -4
    assert lib.spec_tree_probs(C.byref(good_in()), 0, None, None, None, 0, None) == -1


def test_query_plan():
    p = binding.query_plan(128256)
    assert p["cluster_size"] == 8 and p["slice_len"] % 8 == 0 and p["slice_len"] * 8 >= 128256
    assert p["smem_bytes"] <= 113 * 1024 and p["threads"] == 256     # two CTAs per SM
    assert binding.query_plan(1000, 0)["cluster_size"] == 1
    big = binding.query_plan(262144)
    assert big["slice_len"] * big["cluster_size"] >= 262144 and big["smem_bytes"] <= 227 * 1024


def test_binding_refuses_to_run_without_a_gpu():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    z = torch.zeros((1, 2, 8))
    with pytest.raises(RuntimeError):
        binding.tree_probs(z)
    with pytest.raises(RuntimeError):
        binding.sample_bonus(torch.zeros((1, 8)), torch.zeros(1))
