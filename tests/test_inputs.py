"""The seeded input generator: shapes, statistics, determinism."""
import numpy as np

import ppd_inputs


def test_blob_layout_and_statistics(tiny_shape, tiny_blob):
    v = ppd_inputs.blob_views(tiny_shape, tiny_blob)
    assert v["E"].shape == (4096, 256) and v["Wd.3"].shape == (256, 688) and v["Wg.0"].shape == (688, 256)
    for name, std in (("E", 0.02), ("Wq.0", 0.02), ("Wg.2", 0.02), ("W_H", 0.02), ("Wo.1", 0.002), ("Wd.3", 0.002)):
        f = ppd_inputs.bf16_to_f32(v[name]).astype(np.float64)
        n = f.size
        assert abs(f.mean()) < 5 * std / np.sqrt(n)
        assert abs(f.std() / std - 1) < 5 / np.sqrt(2 * n) + 2e-3      # bf16 rounding adds ~1e-3 relative
    assert (ppd_inputs.bf16_to_f32(v["g1.0"]) == 1).all() and (ppd_inputs.bf16_to_f32(v["g_final"]) == 1).all()
    # distinct tensors are distinct draws
    assert not np.array_equal(v["Wq.0"], v["Wk.0"]) and not np.array_equal(v["Wq.0"], v["Wq.1"])


def test_deterministic_and_seeded(tiny_shape, tiny_blob):
    assert np.array_equal(ppd_inputs.gen_weights(tiny_shape, seed=0), tiny_blob)
    assert not np.array_equal(ppd_inputs.gen_weights(tiny_shape, seed=1), tiny_blob)
    p = ppd_inputs.gen_prompt(4096, 1000, seed=1)
    assert np.array_equal(p, ppd_inputs.gen_prompt(4096, 1000, seed=1))
    assert p.min() >= 0 and p.max() < 4096 and len(np.unique(p)) > 800


def test_parameter_counts():
    assert ppd_inputs.LLAMA_7B.blob_elems == 6_738_415_616
    assert ppd_inputs.LLAMA_13B.blob_elems == 13_015_864_320
    assert ppd_inputs.LLAMA_7B.layer_params == 202_383_360
