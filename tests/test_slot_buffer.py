"""Host logic of the fixed-size slot buffer (sliding window, top-S by utility, hybrid); no GPU."""
import pytest

from paper_2603_15619_b200.slots import SlotBuffer


def run(buf, n_layers, utilities):
    """Writes n_layers layers; utilities(layer, owners) -> per-slot utility seen when `layer` is about to be written."""
    history = []
    for layer in range(n_layers):
        slot = buf.next_slot(utilities(layer, list(buf.owner)))
        buf.record(slot, layer)
        history.append((slot, sorted(buf.layers())))
    return history


def test_window_keeps_the_most_recent_layers():
    buf = SlotBuffer(3)
    hist = run(buf, 7, lambda layer, owners: None)
    assert [h[0] for h in hist] == [0, 1, 2, 0, 1, 2, 0]
    assert hist[-1][1] == [4, 5, 6] and buf.filled == 3


def test_top_keeps_the_layers_of_highest_utility():
    worth = {0: 5.0, 1: 0.1, 2: 3.0, 3: 0.2, 4: 9.0, 5: 0.3}          # utility of a layer's slot, constant over time
    buf = SlotBuffer(3, policy="top")
    hist = run(buf, 6, lambda layer, owners: [worth[o] if o is not None else 0.0 for o in owners])
    # full after layer 2 = {0, 1, 2}; layer 3 evicts 1 (0.1); layer 4 evicts 3 (0.2); layer 5 evicts 2 (3.0)
    assert hist[3][1] == [0, 2, 3] and hist[4][1] == [0, 2, 4] and hist[5][1] == [0, 4, 5]


def test_hybrid_protects_the_most_recent_layers():
    worth = {0: 5.0, 1: 4.0, 2: 0.1, 3: 0.05, 4: 0.01, 5: 0.0}
    buf = SlotBuffer(4, policy="hybrid", n_recent=2)
    hist = run(buf, 6, lambda layer, owners: [worth[o] if o is not None else 0.0 for o in owners])
    # layer 4: {0,1,2,3} full, recent {2,3} protected -> evict 1 (4.0 < 5.0); layer 5: {0,2,3,4}, protected {3,4} -> evict 2
    assert hist[4][1] == [0, 2, 3, 4] and hist[5][1] == [0, 3, 4, 5]


def test_ties_go_to_the_oldest_layer_and_bad_arguments_are_refused():
    buf = SlotBuffer(2, policy="top")
    buf.record(buf.next_slot(), 0)
    buf.record(buf.next_slot(), 1)
    assert buf.next_slot([1.0, 1.0]) == 0
    with pytest.raises(ValueError):
        buf.next_slot()                                 # a full utility buffer needs utilities
    with pytest.raises(ValueError):
        SlotBuffer(0)
    with pytest.raises(ValueError):
        SlotBuffer(3, policy="hybrid", n_recent=3)
    with pytest.raises(ValueError):
        SlotBuffer(3, policy="lru")
    fresh = SlotBuffer(3)
    with pytest.raises(ValueError):
        fresh.record(2, 0)                              # free slots are filled in order
