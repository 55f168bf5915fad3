"""The C-ABI library loads and exports every symbol the header declares (no GPU needed)."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "qzo.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(qzo_[a-z0-9_]+)\s*\(", text)))


def test_library_builds_and_exports_header_symbols():
    from paper_2505_13430_b200 import build
    path = build.build()
    lib = ctypes.CDLL(path)
    names = _declared()
    assert len(names) >= 20
    for n in names:
        assert hasattr(lib, n), f"{n} declared in include/qzo.h but not exported"


def test_binding_covers_header_and_host_only_calls_work():
    from paper_2505_13430_b200 import qzo, inputs
    assert sorted(qzo.EXPORTS) == _declared()
    assert qzo._lib.qzo_strerror(0) == b"ok"
    header = open(os.path.join(ROOT, "include", "qzo.h")).read()
    shift = re.search(r"#define QZO_NOALLOC_SCRATCH_BYTES \((\d+)u << (\d+)\)", header)
    assert qzo.NOALLOC_SCRATCH_BYTES == int(shift.group(1)) << int(shift.group(2))
    assert b"workspace" in qzo._lib.qzo_strerror(qzo.ERR_WORKSPACE)
    # host-side queries need no device
    assert qzo.qzo_repacked_bytes(4096, 4096) == 4096 * 4096 // 2
    assert qzo.qzo_repacked_bytes(688, 256) == 2 * 11 * 4096          # padded to 128 x 64 blocks
    assert qzo.qzo_gemm_workspace_bytes(4096, 4096, 4096) == 0
    assert qzo.qzo_gemm_workspace_bytes(16, 4096, 4096) > 0
    flat, train = qzo.qzo_num_scales(inputs.model_cfg("llama7b"))
    assert train == 50_593_792 and flat == train
    assert qzo.qzo_num_scales(inputs.model_cfg("opt6.7b"))[1] == 50_331_648
    assert qzo.qzo_num_scales(inputs.model_cfg("llama13b"))[1] == 99_123_200
    assert qzo.qzo_num_scales(inputs.model_cfg("tiny"))[1] == 12_672
    assert qzo.qzo_scale_layout(inputs.model_cfg("tiny"), 0, 1) == (512, 2, 256)
    assert qzo.qzo_scale_layout(inputs.model_cfg("tiny"), 1, 6) == (6336 + 4 * 512 + 2 * 1376, 6, 256)
    assert qzo.qzo_workspace_bytes(inputs.model_cfg("tiny"), 256) > 0
    bad = dict(inputs.model_cfg("tiny")); bad["n_heads"] = 3
    try:
        qzo.qzo_num_scales(bad)
        assert False
    except qzo.QzoError as e:
        assert e.status == qzo.ERR_BAD_ARG


def test_scale_layout_agrees_with_oracle_inventory():
    from oracle import model as omodel
    from paper_2505_13430_b200 import qzo, inputs
    for name in ("tiny", "tiny_opt", "llama7b", "opt6.7b"):
        cfg = inputs.model_cfg(name)
        bases, total = omodel.scale_index_bases(cfg)
        assert qzo.qzo_num_scales(cfg)[0] == total
        order = omodel.LINEAR_ORDER[cfg["arch"]]
        for layer in (0, cfg["n_layers"] - 1):
            for i, nm in enumerate(order):
                assert qzo.qzo_scale_layout(cfg, layer, i)[0] == bases[layer][nm]
