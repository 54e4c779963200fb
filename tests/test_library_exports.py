"""The C-ABI library builds, loads without a GPU and exports every symbol the header declares."""
import os
import re

from paper_2407_02328_b200 import build


def test_library_exports_every_declared_symbol():
    build.build()
    from paper_2407_02328_b200 import adore
    lib = adore._lib()
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    text = open(os.path.join(root, "include", "adore.h")).read()
    declared = set(re.findall(r"\b(adore_[a-z_0-9]+)\s*\(", text))
    assert declared, "no declarations found"
    for name in sorted(declared):
        assert hasattr(lib, name), f"{name} is declared but not exported"
    assert declared == set(adore.EXPORTS)
    assert adore.adore_status_string(0) == "ok"


def test_create_rejects_bad_arguments_before_touching_the_device():
    from paper_2407_02328_b200 import adore
    import numpy as np
    import workloads as wl
    cfg = wl.get_config(1)
    ctrl = wl.controller_weights(cfg)
    bad = adore.make_config(batch=1, n_layers=1, n_heads=8, head_dim=64, hidden=512, capacity=64, rebuild_max=64,
                            topk=64, max_tokens=256, dtype="f32")
    try:
        adore.adore_cache_create(bad, ctrl)
        assert False, "rebuild_max == capacity must be rejected"
    except adore.AdoreError as e:
        assert e.status == 1
    bad = adore.make_config(batch=1, n_layers=1, n_heads=8, head_dim=48, hidden=512, capacity=64, rebuild_max=8,
                            topk=64, max_tokens=256, dtype="f32")
    try:
        adore.adore_cache_create(bad, ctrl)
        assert False
    except adore.AdoreError as e:
        assert e.status == 8
    adore.adore_cache_destroy(None)
