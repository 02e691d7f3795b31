"""The workload table and the seeded generator (no arithmetic of the method here)."""
import numpy as np

from paper_2511_05534_b200 import configs, inputs


def test_budget_table():
    # (L, B) pairs implied by the five benchmark configurations
    expect = {"cfg1": (192, {250: 48}), "cfg2": (640, {50: 32, 100: 64, 200: 128}), "cfg3": (2176, {100: 218}),
              "cfg4": (8448, {50: 423, 200: 1690}), "cfg5": (33792, {50: 1690})}
    for name, (L, table) in expect.items():
        wl = configs.get(name)
        assert wl.seq_len == L
        for pm, B in table.items():
            assert wl.n_keep(pm) == B
    assert configs.get("cfg5").n_units == 320 and configs.get("cfg3").group == 7


def test_generator_is_seeded_and_shaped():
    wl = configs.get("cfg2")
    a = inputs.make_unit(wl, 3)
    b = inputs.make_unit(wl, 3)
    c = inputs.make_unit(wl, 4)
    assert all(np.array_equal(a[key], b[key]) for key in a)
    assert not np.array_equal(a["k"], c["k"])
    assert a["q"].shape == (32, 32, 128) and a["k"].shape == (32, 640, 128) and a["modality"].sum() == 576
    # bf16 workloads hold bf16-representable values only
    assert np.all((a["k"].view(np.uint32) & 0xFFFF) == 0)
    vis = a["modality"] == 1
    assert abs(a["v"][:, vis].mean() - 0.5) < 0.02 and abs(a["v"][:, ~vis].mean()) < 0.02


def test_round_to_bf16_ties_to_even():
    x = np.array([1.0, 1.0 + 2 ** -8, 1.0 + 3 * 2 ** -8, 1.0 + 2 ** -7], dtype=np.float32)
    assert inputs.round_to_bf16(x).tolist() == [1.0, 1.0, 1.0 + 2 ** -6, 1.0 + 2 ** -7]


def test_video_window_is_mixed_modality():
    wl = configs.get("cfg4")
    m = inputs.modality_map(wl)
    assert m[-64:].tolist() == [1] * 32 + [0] * 32
