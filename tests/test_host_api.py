"""CPU-only checks of the C ABI: the library loads, exports every declared symbol, and its
host-side validation and size queries behave as the header says.  No kernel runs here."""
import ctypes as C
import os
import re

import pytest
import torch

import c2t_inputs
import paper_2502_13652_b200 as c2t
from paper_2502_13652_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    build.build()
    return c2t.lib()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "c2t.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(c2t_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(L):
    names = declared_symbols()
    assert {"c2t_init", "c2t_expand_level", "c2t_prune", "c2t_build_verify", "c2t_accept"} <= set(names)
    for name in names:
        assert hasattr(L, name), f"{name} declared in include/c2t.h but not exported"


def cfg(**kw):
    w = c2t_inputs.classifier_weights(16)
    base = dict(batch=2, vocab=1000, dtype=c2t.F32, max_depth=4, topk=5, frontier_cap=5, budget=20,
                threshold=0.5, hidden=16, w1=w[0], b1=w[1], w2=w[2], b2=w[3])
    base.update(kw)
    return c2t.Config(**base)


def test_sizes(L):
    c = cfg()
    assert c2t.c2t_tree_capacity(c) == 1 + 5 + 3 * 5
    assert c2t.c2t_final_width(c) == 20
    assert c2t.c2t_mask_words(c) == 1
    assert c2t.c2t_final_width(cfg(budget=0)) == 21
    assert c2t.c2t_final_width(cfg(budget=80, max_depth=10, topk=8, frontier_cap=16)) == 80
    assert c2t.c2t_mask_words(cfg(budget=80, max_depth=10, topk=8, frontier_cap=16)) == 2
    assert c2t.c2t_tree_capacity(cfg(tree_add=c2t.ADD_ALL_SURVIVORS, max_depth=11, topk=10, frontier_cap=10)) == 1011
    assert c2t.c2t_workspace_bytes(c) > 0
    assert c2t.c2t_workspace_bytes(c) % 256 == 0
    assert c2t.c2t_workspace_bytes(cfg(batch=64)) > c2t.c2t_workspace_bytes(c)


@pytest.mark.parametrize("bad,code", [
    (dict(batch=0), c2t.EINVAL), (dict(vocab=0), c2t.EINVAL), (dict(dtype=7), c2t.EINVAL),
    (dict(classifier=3), c2t.EINVAL), (dict(tree_add=2), c2t.EINVAL), (dict(entropy_top_m=-1), c2t.EINVAL),
    (dict(w1=None), c2t.EINVAL), (dict(threshold=float("nan")), c2t.EINVAL),
    (dict(topk=33), c2t.ERANGE), (dict(frontier_cap=33), c2t.ERANGE), (dict(hidden=65), c2t.ERANGE),
    (dict(budget=1025), c2t.ERANGE), (dict(batch=4097), c2t.ERANGE), (dict(max_depth=33), c2t.ERANGE),
    (dict(tree_add=c2t.ADD_ALL_SURVIVORS, topk=32, frontier_cap=32, max_depth=10), c2t.ERANGE),
])
def test_init_rejects_bad_configurations(L, bad, code):
    c = cfg(**bad)
    s, keep = c.c_struct()
    assert L.c2t_workspace_bytes(C.byref(s)) == 0
    handle = C.c_void_p()
    buf = (C.c_char * 512)()
    addr = (C.addressof(buf) + 255) & ~255
    assert L.c2t_init(C.byref(s), addr, 1 << 40, C.byref(handle)) == code
    assert not handle


def test_init_checks_workspace_before_touching_cuda(L):
    c = cfg()
    s, keep = c.c_struct()
    handle = C.c_void_p()
    need = L.c2t_workspace_bytes(C.byref(s))
    assert L.c2t_init(C.byref(s), None, need, C.byref(handle)) == c2t.EINVAL
    assert L.c2t_init(C.byref(s), 256 + 8, need, C.byref(handle)) == c2t.EALIGN
    assert L.c2t_init(C.byref(s), 256, need - 1, C.byref(handle)) == c2t.ERANGE
    assert L.c2t_init(C.byref(s), 256, need, None) == c2t.EINVAL


@pytest.mark.skipif(torch.cuda.is_available(), reason="checks the loud failure on a box without a GPU")
def test_init_fails_loudly_without_a_gpu(L):
    c = cfg()
    s, keep = c.c_struct()
    handle = C.c_void_p()
    need = L.c2t_workspace_bytes(C.byref(s))
    assert L.c2t_init(C.byref(s), 256, need, C.byref(handle)) == c2t.ECUDA
    assert not handle


def test_null_context_is_rejected(L):
    assert L.c2t_begin_step(None, None, None, None) == c2t.EINVAL
    assert L.c2t_expand_level(None, 0, None, 0, 0, None) == c2t.EINVAL
    assert L.c2t_prune(None, 0, None, None) == c2t.EINVAL
    assert L.c2t_build_verify(None, None, None) == c2t.EINVAL
    assert L.c2t_accept(None, None, 0, 0, None, None) == c2t.EINVAL
    assert L.c2t_launch_count(None) == 0


def test_strerror(L):
    assert L.c2t_strerror(0) == b"ok"
    seen = {L.c2t_strerror(code) for code in (0, -1, -2, -3, -4, -5, -6)}
    assert len(seen) == 7
    assert L.c2t_strerror(-99) == b"unknown error"


def test_struct_layouts_match_the_header():
    # field order of the ctypes mirrors follows the header; a reordering would break every call
    text = open(os.path.join(ROOT, "include", "c2t.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    for struct, mirror in (("c2t_frontier", binding.c2t_frontier), ("c2t_verify", binding.c2t_verify),
                           ("c2t_accept_out", binding.c2t_accept_out), ("c2t_config", binding.c2t_config),
                           ("c2t_host_step", binding.c2t_host_step)):
        body = re.search(r"typedef struct \{([^{}]*)\} " + struct + ";", text).group(1)
        names = []
        for decl in body.split(";"):
            decl = decl.strip()
            if not decl:
                continue
            for part in decl.split(","):
                names.append(re.findall(r"([A-Za-z_0-9]+)\s*$", part.strip())[0])
        assert names == [n for n, _ in mirror._fields_], struct


def test_classifier_weights_file_round_trip(tmp_path):
    """save_classifier / load_classifier keep every float32 bit and refuse damaged files."""
    import c2t_inputs
    from paper_2502_13652_b200 import save_classifier, load_classifier
    w = c2t_inputs.classifier_weights(48, seed=3)
    path = str(tmp_path / "ffn.c2tw")
    save_classifier(path, *w)
    back = load_classifier(path)
    for a, b in zip(w, back):
        assert a.dtype == b.dtype == torch.float32 and a.shape == b.shape and torch.equal(a, b)
    blob = open(path, "rb").read()
    for bad in (blob[:-4], b"X" + blob[1:], blob + b"\0\0\0\0"):
        open(path, "wb").write(bad)
        with pytest.raises(ValueError):
            load_classifier(path)
    with pytest.raises(ValueError):
        save_classifier(path, torch.zeros(65, 3), torch.zeros(65), torch.zeros(65), torch.zeros(1))
