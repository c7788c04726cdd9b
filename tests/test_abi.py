"""Host-side checks that need no GPU: the library builds, loads, and exports what the header declares."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2603_16219_b200 import binding, build
    build.build()
    return binding.load_library()


def _declared_symbols():
    names = set()
    inc = os.path.join(ROOT, "include")
    for f in os.listdir(inc):
        if f.endswith(".h"):
            txt = open(os.path.join(inc, f)).read()
            txt = re.sub(r"/\*.*?\*/", "", txt, flags=re.S)
            names |= set(re.findall(r"\b(specsteer_[a-z_0-9]+)\s*\(", txt))
    return names


def test_every_declared_symbol_is_exported(lib):
    from paper_2603_16219_b200 import binding
    declared = _declared_symbols()
    assert declared, "no declarations found"
    assert declared == set(binding.EXPORTS)
    for name in declared:
        assert getattr(lib, name) is not None


def test_version_and_status_strings(lib):
    assert lib.specsteer_version() >= 0x000100
    seen = {lib.specsteer_status_string(i).decode() for i in range(7)}
    assert len(seen) == 7 and "ok" in seen
    assert lib.specsteer_status_string(99).decode() == "unknown status"


def test_descriptor_layout_matches_header(lib):
    """The ctypes mirror must have the header's field order and a size the C compiler agrees with."""
    from paper_2603_16219_b200 import binding
    hdr = open(os.path.join(ROOT, "include", "specsteer.h")).read()
    body = hdr[hdr.index("typedef struct {"):hdr.index("} specsteer_round_desc;")]
    body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
    fields = []
    for decl in body.split(";"):
        decl = decl.replace("typedef struct {", "").strip()
        if not decl:
            continue
        for part in decl.split(","):
            fields.append(re.findall(r"([A-Za-z_0-9]+)\s*$", part.strip())[0])
    mirror = [n for n, _ in binding.RoundDesc._fields_]
    assert [f if f != "lambda" else "lam" for f in fields] == mirror
    assert C.sizeof(binding.RoundDesc) == 3 * 4 + 4 + 2 * 8 + 4 * 4 + 23 * 8


def test_host_checkable_errors_launch_nothing(lib):
    """NULL context / descriptor are rejected before any CUDA call is made."""
    from paper_2603_16219_b200 import binding
    d = binding.RoundDesc()
    assert lib.specsteer_verify_round(None, C.byref(d), None) == binding.ERR_INVALID_ARG
    assert lib.specsteer_recover_sample(None, C.byref(d), None) == binding.ERR_INVALID_ARG
    assert lib.specsteer_round_host(None, C.byref(d), None) == binding.ERR_INVALID_ARG
    assert lib.specsteer_ctx_destroy(None) == binding.ERR_INVALID_ARG
    assert lib.specsteer_ctx_create(None, 0, 1, 1, 1) == binding.ERR_INVALID_ARG
    h = C.c_void_p()
    assert lib.specsteer_ctx_create(C.byref(h), 0, 0, 1, 1) == binding.ERR_INVALID_ARG
    assert lib.specsteer_ctx_workspace_bytes(None) == 0


def test_product_has_no_cpu_fallback_and_never_imports_the_oracle():
    import torch
    from paper_2603_16219_b200 import binding
    if not torch.cuda.is_available():
        with pytest.raises(RuntimeError):
            binding.Context(1, 1, 8)
    pkg = os.path.join(ROOT, "paper_2603_16219_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                txt = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in txt.replace("the CPU oracle", ""), f


def test_lmhead_descriptor_marshalling_rejects_bad_operands():
    """Host-side checks of the LM-head descriptor builder (no GPU: only shapes, dtypes and pointers are looked at)."""
    import torch
    from paper_2603_16219_b200 import binding as b
    B, K, V, dL, dS = 2, 3, 40, 16, 8
    bf = torch.bfloat16
    inputs = {
        "x_llm": torch.zeros(B, K + 1, dL, dtype=bf), "w_llm": torch.zeros(V, dL, dtype=bf),
        "x_slm_plus": torch.zeros(B, K + 1, dS, dtype=bf), "w_slm_plus": torch.zeros(V, dS, dtype=bf),
        "x_slm_minus": torch.zeros(B, K + 1, dS, dtype=bf), "w_slm_minus": torch.zeros(V, dS, dtype=bf),
        "draft_tokens": torch.zeros(B, K, dtype=torch.int32), "draft_len": torch.zeros(B, dtype=torch.int32),
        "lam": torch.ones(B), "beta": torch.ones(B), "temperature": torch.ones(B),
        "u_accept": torch.zeros(B, K), "u_recover": torch.zeros(B),
    }
    outs = b.alloc_outputs(B, K, "cpu")
    d = b.make_lmhead_desc(inputs, outs, flags=b.FLAG_BONUS)
    assert (d.round.B, d.round.K, d.round.V, d.d_llm, d.d_slm) == (B, K, V, dL, dS)
    assert d.x_llm == inputs["x_llm"].data_ptr() and d.w_slm_minus == inputs["w_slm_minus"].data_ptr()
    assert d.round.accept_len == outs["accept_len"].data_ptr() and d.round.flags == b.FLAG_BONUS
    import pytest
    for key, bad in (("w_llm", torch.zeros(V, dL)),                       # float32 head
                     ("x_slm_plus", torch.zeros(B, K + 1, dS + 8, dtype=bf)),  # width differs from its head
                     ("w_slm_minus", torch.zeros(V + 1, dS, dtype=bf)),        # vocabulary differs
                     ("x_llm", torch.zeros(B, K + 1, 2 * dL, dtype=bf)[..., ::2])):  # not contiguous
        broken = dict(inputs)
        broken[key] = bad
        with pytest.raises(ValueError):
            b.make_lmhead_desc(broken, outs)
    broken = dict(inputs)
    broken["beta"] = torch.ones(B + 1)
    with pytest.raises(ValueError):
        b.make_lmhead_desc(broken, outs)


def test_lmhead_descriptor_layout_matches_header(lib):
    from paper_2603_16219_b200 import binding
    hdr = open(os.path.join(ROOT, "include", "specsteer.h")).read()
    end = hdr.index("} specsteer_lmhead_desc;")
    body = re.sub(r"/\*.*?\*/", "", hdr[hdr.rindex("typedef struct {", 0, end):end], flags=re.S)
    fields = []
    for decl in body.split(";"):
        decl = decl.replace("typedef struct {", "").strip()
        if not decl:
            continue
        for part in decl.split(","):
            fields.append(re.findall(r"([A-Za-z_0-9]+)\s*$", part.strip())[0])
    assert fields == [n for n, _ in binding.LmheadDesc._fields_]
    assert C.sizeof(binding.LmheadDesc) == C.sizeof(binding.RoundDesc) + 6 * 8 + 2 * 4 == 288
