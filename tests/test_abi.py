"""The C-ABI library loads without a GPU and exports every symbol the header declares; host-side
configuration checks run without touching the device."""
import os
import re

import pytest

import synth
import paper_2603_17942_b200 as P
from paper_2603_17942_b200 import build as esp_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    esp_build.build()
    return P.load_library()


def _declared():
    text = open(os.path.join(ROOT, "include", "esp.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(esp_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared()
    assert len(names) >= 14
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(P.EXPORTS) == names


def test_binding_mirrors_the_header():
    """The constants and the struct members of the ctypes mirror are the header's, in the header's order."""
    import ctypes
    text = open(os.path.join(ROOT, "include", "esp.h")).read()
    for name, value in (("ESP_MAX_ROWS", P.ESP_MAX_ROWS), ("ESP_MAX_PROBES", P.ESP_MAX_PROBES),
                        ("ESP_MAX_KPRIME", P.ESP_MAX_KPRIME), ("ESP_MAX_UNREAD_STEPS", P.ESP_MAX_UNREAD_STEPS),
                        ("ESP_PREFILL_CHUNK", P.ESP_PREFILL_CHUNK)):
        m = re.search(r"#define\s+%s\s+(\d+)" % name, text)
        assert m and int(m.group(1)) == value, name
    m = re.search(r"#define\s+ESP_STATIC_SCRATCH_BYTES\s+\((\d+)u\s*<<\s*(\d+)\)", text)
    assert m and (int(m.group(1)) << int(m.group(2))) == P.ESP_STATIC_SCRATCH_BYTES
    code = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    for cname, ctype in (("esp_model_cfg", P.esp_model_cfg), ("esp_spec_cfg", P.esp_spec_cfg), ("esp_stats", P.esp_stats)):
        end = code.index("} %s;" % cname)
        body = code[code.rindex("typedef struct {", 0, end) + len("typedef struct {"):end]
        members = []
        for decl in body.split(";"):
            decl = decl.strip()
            if not decl:
                continue
            names = decl.split(None, 1)[1]
            members += [n.strip().split("[")[0] for n in names.split(",")]
        mirror = [f[0] for f in ctype._fields_]
        assert [("lam" if n == "lambda" else n) for n in members] == mirror, cname
    # two floats, two 32-bit seed words and the 32-bit members: no padding anywhere
    assert ctypes.sizeof(P.esp_spec_cfg) == 4 * (len(P.esp_spec_cfg._fields_) - 1 + P.ESP_MAX_PROBES)


def test_workspace_bytes_and_config_checks(lib):
    m = P.model_cfg(synth.LLAMA3_8B, 1024 + 256 + 16)
    s = P.spec_cfg(n_probes=4, topk=10, max_nodes=64, expand_width=0, n_anchor=1)
    nbytes = P.esp_workspace_bytes(m, s)
    kv = 2 * 32 * 8 * (1296 + P.ESP_MAX_ROWS) * 128 * 2
    packed = synth.LLAMA3_8B.n_params_streamed() * 2       # the streaming copy of every layer matrix and the LM head
    assert kv + packed <= nbytes < kv + packed + (1 << 30)
    # the paper's operating points fit: k=1 with a 30-node tree, k=2 with a 20-node tree (60 rows each)
    for k, B in ((1, 30), (2, 20)):
        P.esp_workspace_bytes(m, P.spec_cfg(n_probes=k, topk=14, max_nodes=B, n_anchor=0))
    # static trees: [7,2] and [15,4] with a mask pair per node are 30 and 60 rows
    for widths in ((7, 2), (15, 4), (14,)):
        P.esp_workspace_bytes(m, P.spec_cfg(n_probes=len(widths), n_anchor=0, static_widths=widths))
    bad = [P.spec_cfg(n_probes=4, topk=10, max_nodes=64, n_anchor=0),      # (k+1)*64 rows > 128
           P.spec_cfg(n_probes=3, n_anchor=0, static_widths=(7, 5, 20)),   # (k+1)*(1+32) rows > 128
           P.spec_cfg(n_probes=2, n_anchor=1, static_widths=(40, 2)),      # K' beyond the kept list length
           P.spec_cfg(n_probes=9, topk=4, max_nodes=8),                    # too many probes
           P.spec_cfg(n_probes=2, topk=40, max_nodes=8),                   # K' beyond the kept list length
           P.spec_cfg(n_probes=2, topk=0, max_nodes=8)]
    for sp in bad:
        with pytest.raises(P.EspError) as e:
            P.esp_workspace_bytes(m, sp)
        assert e.value.code == -1
    with pytest.raises(P.EspError):
        P.esp_workspace_bytes(P.model_cfg(synth.LLAMA3_8B.replace(n_kv_heads=7), 128), s)
    with pytest.raises(P.EspError):
        P.esp_workspace_bytes(P.model_cfg(synth.LLAMA3_8B.replace(head_dim=96), 128), s)


def test_missing_library_fails_loudly(tmp_path):
    with pytest.raises(OSError):
        P.load_library(str(tmp_path / "nope.so"))
