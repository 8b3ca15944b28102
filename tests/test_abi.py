"""The C-ABI library loads without a GPU and exports every symbol the header declares."""
import ctypes
import os
import re

import pytest

from paper_1712_01670_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "deepcache.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(dc_[a-z_]+)\s*\(", text)))


def test_library_builds_and_exports_header_symbols():
    lib = ctypes.CDLL(build.build())
    names = declared_symbols()
    assert len(names) >= 15
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in deepcache.h but not exported"
    assert sorted(binding.EXPORTS) == names


def test_struct_layouts_match_the_header():
    assert ctypes.sizeof(binding.dc_region) == 24
    assert ctypes.sizeof(binding.dc_layer_desc) == 60
    assert ctypes.sizeof(binding.dc_config) == 88 and binding.dc_config.psnr_db.offset == 40
    assert binding.dc_config.region_mode.offset == 56
    assert ctypes.sizeof(binding.dc_frame_stats) == 7 * 4 + 4 * binding.DC_MAX_LAYERS


def test_status_strings_and_argument_errors_without_gpu():
    assert binding.strerror(binding.DC_OK) == "ok"
    assert "rectangles" in binding.strerror(binding.DC_ERR_OVERFLOW)
    lib = binding.load()
    # null arguments and bad configurations are rejected before any CUDA call
    assert lib.dc_cache_create(None, None, 0, None, None, None, None) == binding.DC_ERR_ARG
    cfg = binding.dc_config(width=64, height=64, channels=4, n_streams=1, block=8, range=4, search=1, skip_k=1,
                            expire_n=10, psnr_db=20.0, dtype=0, max_regions=0)
    layers = binding.make_layers([dict(kind=0, kh=3, kw=3, sh=1, sw=1, ph=1, pw=1, cin=3, cout=16, relu=1,
                                       in0=-1, in1=-1, out_h=64, out_w=64)])
    out = ctypes.c_void_p()
    assert lib.dc_cache_create(ctypes.byref(cfg), layers, 1, None, None, None, ctypes.byref(out)) == binding.DC_ERR_CONFIG
    cfg.channels = 3
    layers[0].out_w = 63                                  # inconsistent output size
    assert lib.dc_cache_create(ctypes.byref(cfg), layers, 1, None, None, None, ctypes.byref(out)) == binding.DC_ERR_CONFIG
    assert lib.dc_cache_destroy(None) == binding.DC_ERR_ARG
    assert lib.dc_infer_frame(None, None, 0, None, None) == binding.DC_ERR_ARG


def test_engine_refuses_to_run_without_cuda():
    import torch
    if torch.cuda.is_available():
        pytest.skip("CUDA present")
    from paper_1712_01670_b200.engine import DeepCache
    from paper_1712_01670_b200.synth import configs
    with pytest.raises(RuntimeError):
        DeepCache.from_workload(configs.WORKLOADS[1]())
