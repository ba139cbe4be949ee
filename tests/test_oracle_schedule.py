"""Pins of the schedule oracle against the counts the paper states (Section 3, Section 3.4)."""
from oracle import schedule_oracle as so


def _layers(kind, L, step, **kw):
    return [l + 1 for l in range(L) if so.approximated(kind, L, l, step, **kw)]


def test_first_schedule_counts_match_the_paper():
    # Section 3: the first schedule approximates four layers of VGG-19 and five of ResNet-20
    for step in range(4):
        assert _layers(so.EVERY_4TH_LAYER, 19, step) == [2, 6, 10, 14, 18]
        assert _layers(so.EVERY_4TH_LAYER, 16, step) == [2, 6, 10, 14]


def test_two_layer_cnn_every_other_batch():
    assert [_layers(so.LAYER2_ALT_BATCH, 2, t) for t in range(4)] == [[], [2], [], [2]]


def test_schedules_2_and_3_approximate_a_quarter_of_layer_batches():
    L, T = 20, 8
    for kind in (so.ALT_LAYER_ALT_BATCH, so.ALL_LAYERS_EVERY_4TH_BATCH):
        hits = sum(so.approximated(kind, L, l, t) for l in range(L) for t in range(T))
        assert hits * 4 == L * T
    assert _layers(so.ALL_LAYERS_EVERY_4TH_BATCH, 5, 3) == [1, 2, 3, 4, 5]
    assert _layers(so.ALT_LAYER_ALT_BATCH, 5, 1) == [2, 4] and _layers(so.ALT_LAYER_ALT_BATCH, 5, 2) == []


def test_splitmix64_first_outputs_of_the_zero_seeded_stream():
    # the generator's state advances by the golden-ratio increment; output t mixes state t+1 increments
    inc = 0x9E3779B97F4A7C15
    outs = [so.splitmix64((t * inc) & (2 ** 64 - 1)) for t in range(3)]
    assert outs == [0xE220A8397B1DCDAF, 0x6E789E6AA1B965F4, 0x06C45D188009454F]


def test_seeded_fraction_masks():
    for L in (16, 19):
        for f, m in ((0.0, 0), (0.25, int(0.25 * L + 0.5)), (0.5, int(0.5 * L + 0.5)), (0.75, int(0.75 * L + 0.5)), (1.0, L)):
            mask = so.fraction_mask(L, f, 1234)
            assert sum(mask) == m
            assert _layers(so.SEEDED_FRACTION_ALT_BATCH, L, 0, fraction=f, seed=1234) == []
            assert _layers(so.SEEDED_FRACTION_ALT_BATCH, L, 1, fraction=f, seed=1234) == [l + 1 for l in range(L) if mask[l]]
    assert so.fraction_mask(19, 0.5, 1) != so.fraction_mask(19, 0.5, 2)
    # nested: a larger fraction keeps the layers of a smaller one (same hash order)
    small = so.fraction_mask(19, 0.25, 9); big = so.fraction_mask(19, 0.75, 9)
    assert all(b or not s for s, b in zip(small, big))
