"""Host-side checks of the C-ABI library that need no GPU: it loads, exports
every declared entry point, validates configurations, and its manifest and
workspace plan are consistent."""
import ctypes as C
import os
import re

import pytest

from paper_2203_17189_b200 import binding as Bd
from paper_2203_17189_b200 import build as builder
from paper_2203_17189_b200 import workloads as WL

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built():
    builder.build()


def test_exports_every_declared_symbol():
    hdr = open(os.path.join(ROOT, "include", "t5_b200.h")).read()
    declared = re.findall(r"T5_API\s+[\w\s\*]+?\b(t5_\w+)\s*\(", hdr)
    assert len(declared) >= 15
    L = Bd.lib()
    for name in declared:
        assert hasattr(L, name), name
    assert sorted(declared) == sorted(Bd.EXPORTS)


def test_manifest_layout():
    dims = WL.model_dims("tiny")
    h = Bd.Handle(Bd.make_config(dims, 4, 64, 32, "f32"))
    man = h.t5_param_manifest()
    names = [m[0] for m in man]
    assert names[0] == "token_embed" and "enc.relbias" in names and "dec.L1.cross.o" in names
    total = h.t5_param_count()
    end = 0
    for name, off, shape in man:
        assert off % 64 == 0 and off >= end
        n = 1
        for s in shape:
            n *= s
        end = off + n
    assert end <= total
    d = dict((m[0], m) for m in man)
    # q, k, v of a block are contiguous so they form one [3I, d] matrix
    q, k, v = d["enc.L0.attn.q"], d["enc.L0.attn.k"], d["enc.L0.attn.v"]
    assert k[1] == q[1] + 128 * 128 and v[1] == k[1] + 128 * 128
    assert d["enc.L0.ffn.wi1"][1] == d["enc.L0.ffn.wi0"][1] + 256 * 128
    assert d["enc.L0.attn.q"][2] == (128, 128) and d["enc.L0.ffn.wo"][2] == (128, 256)
    assert h.t5_workspace_bytes() > 0
    # decoder-only has no encoder / cross tensors
    h2 = Bd.Handle(Bd.make_config(WL.model_dims("declm", n_dec_layers=2), 1, 0, 64, "bf16"))
    n2 = [m[0] for m in h2.t5_param_manifest()]
    assert not any(n.startswith("enc.") or ".cross." in n for n in n2)


@pytest.mark.parametrize("field,value", [("d_kv", 48), ("d_model", 100), ("arch", 2), ("dtype", 3),
                                         ("n_dec_layers", 0), ("abi_version", 99), ("rel_buckets", 6),
                                         ("vocab", 1001)])
def test_bad_config_is_rejected(field, value):
    cfg = Bd.make_config(WL.model_dims("tiny"), 4, 64, 32, "f32")
    setattr(cfg, field, value)
    with pytest.raises(Bd.T5Error) as e:
        Bd.Handle(cfg)
    assert e.value.code == -2


def test_null_arguments():
    L = Bd.lib()
    assert L.t5_create(None, None) == -1
    n = C.c_int64()
    assert L.t5_param_count(None, C.byref(n)) == -1
    assert L.t5_relpos_buckets(1, 32, 128, 0, 4, None, None) == -1
