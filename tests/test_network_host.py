"""Host-side scheduling of a layer list over CUDA streams (no GPU needed): every layer must wait for all of
its producers that run on another stream, and independent branches must land on different streams."""
from paper_1805_08691_b200 import network
from tests.test_oracle_network import _mini_inception
from workloads import nets


class _Host:
    """The part of QuantNetwork that _assign_streams touches."""

    def __init__(self, layers):
        self.layers = layers
        self.by_name = {L.name: L for L in layers}


def _assign(layers, limit):
    h = _Host(layers)
    network.QuantNetwork._assign_streams(h, limit)
    return h


def test_single_stream_keeps_list_order():
    h = _assign(_mini_inception(), 1)
    assert h.n_streams == 1 and set(h.stream_of.values()) == {0}


def test_branches_get_their_own_streams_and_every_input_is_a_dependency():
    layers = _mini_inception()
    h = _assign(layers, 4)
    s = h.stream_of
    # the three readers of the stem output open three different streams; a chain stays on its stream
    assert len({s["m0_1x1"], s["m0_reduce"], s["m0_pool"]}) == 3
    assert s["m0_proj"] == s["m0_pool"] and s["m0_1x3"] == s["m0_reduce"] and s["m0_3x1"] != s["m0_1x3"]
    # a reader of a concat waits for every member, nested ones included, and for the concat's own copies
    assert set(h.deps["m1_3x3_s2"]) == {"m0_1x1", "m0_1x3", "m0_3x1", "m0_pair", "m0_proj", "m0"}
    assert set(h.deps["m1"]) == {"m1_3x3_s2", "m1_pool"}
    # every tensor a layer reads (directly or through a concat) precedes it and is listed
    seen = {"input"}
    for L in layers:
        for t in h.deps[L.name]:
            assert t in seen, (L.name, t)
        for t in list(L.src) + ([L.residual] if L.residual else []):
            assert t in h.deps[L.name]
        seen.add(L.name)


def test_residual_and_heads():
    h = _assign(nets.bottleneck_stack(C=16, blocks=2), 4)
    assert h.stream_of["blk0_branch1"] != h.stream_of["blk0_branch2a"]          # projection beside the branch
    assert set(h.deps["blk0_branch2c"]) == {"blk0_branch2b", "blk0_branch1"}     # the sum waits for both
    h = _assign(nets.ssd300(), 4)
    assert h.stream_of["conv4_3_mbox_loc"] != h.stream_of["pool4"] and h.n_streams >= 3
