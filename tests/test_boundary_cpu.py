"""CPU-only checks of the boundary: the shared library loads, exports every declared symbol, and the
host-side descriptor logic (workspace sizes, validation order) behaves."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def api():
    import paper_1909_09577_b200 as api
    from paper_1909_09577_b200 import build
    build.build()
    return api


def declared_symbols():
    names = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if not fn.endswith(".h"):
            continue
        src = open(os.path.join(ROOT, "include", fn)).read()
        src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
        for m in re.finditer(r"^\s*(?:int|void|int64_t|const char\*)\s+(\w+)\s*\(", src, flags=re.M):
            names.add(m.group(1))
    return names


def test_library_exports_every_declared_symbol(api):
    lib = api.load_library()
    names = declared_symbols()
    assert {"sepconv_fwd", "sepconv_bwd", "encoder_fwd_bwd", "sepconv_ctx_create"} <= names
    for n in names:
        assert hasattr(lib, n), n


def test_strerror_and_workspace_sizes(api):
    import synth_inputs as si
    assert api.strerror(0) == "ok"
    assert "transposed" in api.strerror(-4)
    d = api.block_desc(si.config(2).layers[0], 32, 400, "f16")
    f, b = api.sepconv_workspace_bytes(d)
    assert f > 0 and b > 32 * 256 * 400 * 2
    d.K = 4                                     # even K is a supported variant
    assert api.sepconv_workspace_bytes(d)[0] > 0
    d.K = 0
    with pytest.raises(api.SepconvError) as e:
        api.sepconv_workspace_bytes(d)
    assert e.value.code == -6
    d.K, d.stride = 33, 3
    with pytest.raises(api.SepconvError):
        api.sepconv_workspace_bytes(d)


def test_encoder_spec_layout(api):
    import synth_inputs as si
    spec = api.EncoderSpec(si.quartznet5x5_layers(), 32, 1600, "bf16")
    assert spec.T_out == 800 and spec.C_out == 29
    n = api.encoder_workspace_bytes(spec)
    assert 1 << 30 < n < 4 << 30
    offs = [o for o in spec.param_offsets if o >= 0]
    assert offs == sorted(offs) and all(o % 256 == 0 for o in offs)
    # identity residual with a channel change is rejected on the host
    bad = [si.LayerCfg(8, 16, K=3, residual="identity")]
    with pytest.raises(api.SepconvError):
        api.encoder_workspace_bytes(api.EncoderSpec(bad, 2, 32, "f32"))


def test_residual_spans_may_overlap_but_not_point_forward(api):
    """Disjoint spans share one pending-gradient buffer; nested spans and shared sources take more workspace;
    a residual from a later layer is refused."""
    import synth_inputs as si
    plain = si.LayerCfg(8, 8, K=3)
    def res(j):
        return si.LayerCfg(8, 8, K=3, residual="identity", res_from=j)
    def bytes_of(layers):
        return api.encoder_workspace_bytes(api.EncoderSpec(layers, 2, 32, "f32"))
    disjoint = bytes_of([plain, plain, res(1), plain, res(3), plain])
    nested = bytes_of([plain, plain, plain, res(2), plain, res(1)])          # [2,3] inside [1,5]
    shared = bytes_of([plain, plain, res(1), res(1), plain, plain])          # two layers share source 1
    assert 0 < disjoint < nested and disjoint < shared
    with pytest.raises(api.SepconvError) as e:
        bytes_of([plain, res(2), plain])
    assert e.value.code == -6


def test_missing_library_fails_loudly(api, tmp_path):
    from paper_1909_09577_b200 import binding
    old = binding._lib
    binding._lib = None
    try:
        with pytest.raises(FileNotFoundError):
            binding.load_library(str(tmp_path / "nope.so"))
    finally:
        binding._lib = old
