"""Schedule generators (inputs to the layer, Sec. 4.2): legality of every order they produce, and the oracle's
split == full-backward equality under the two-chunk orders."""
import numpy as np
import pytest

from harness import c1_inputs, state_equal
from oracle.layer import OracleLinear
from paper_2609_23536_b200 import inputs
from paper_2609_23536_b200.schedules import (full_backward, full_backward_chunks, interleaved_1f1b, peak_live,
                                             peak_live_per_chunk, sched, zb_v)


def _check_legal(s, M, chunks):
    pos = {}
    for i, (a, m, c) in enumerate(s):
        assert 0 <= m < M and 0 <= c < chunks and (a, m, c) not in pos
        pos[(a, m, c)] = i
    assert len(s) == 3 * M * chunks
    for m in range(M):
        for c in range(chunks):
            assert pos[("F", m, c)] < pos[("dI", m, c)] < pos[("dW", m, c)]
    for c in range(chunks):  # a chunk's weight gradients accumulate in microbatch order
        order = [m for a, m, cc in s if a == "dW" and cc == c]
        assert order == sorted(order)


@pytest.mark.parametrize("M,stages", [(4, 2), (8, 4), (12, 4), (16, 8)])
@pytest.mark.parametrize("defer", [0, 2])
def test_interleaved_1f1b_orders_are_legal(M, stages, defer):
    for stage in range(stages):
        s = interleaved_1f1b(M, stages, stage, 2, defer)
        _check_legal(s, M, 2)
        warm = 0
        while s[warm][0] == "F":
            warm += 1
        # warm-up forwards, plus the first forward of the steady phase
        assert warm == min((stages - stage - 1) * 2 + stages, 2 * M) + (1 if (stages - stage - 1) * 2 + stages < 2 * M else 0)
        # the last stage's first backward unit is the LAST chunk of microbatch 0
        assert next(x for x in s if x[0] == "dI") == ("dI", 0, 1)
    with pytest.raises(ValueError):
        interleaved_1f1b(6, 4, 0)


@pytest.mark.parametrize("M,stages", [(4, 2), (8, 4), (6, 3)])
def test_zb_v_orders_are_legal_and_bounded(M, stages):
    for stage in range(stages):
        s = zb_v(M, stages, stage)
        _check_legal(s, M, 2)
        assert sum(peak_live_per_chunk(s)) <= 2 * 2 * stages  # the simulation's live-tape limit (both pools)
        # on the last device the two chunks are adjacent model parts: chunk 1's forward follows chunk 0's directly
        if stage == stages - 1:
            assert s[0] == ("F", 0, 0) and s[1] == ("F", 0, 1)
    # the first device starts the pipeline alone and runs ahead by the depth of the V
    s0 = zb_v(M, stages, 0)
    first_c1 = next(i for i, x in enumerate(s0) if x[2] == 1)
    assert first_c1 >= min(M, 2 * stages - 1)


def test_single_chunk_generator_matches_its_docstring():
    assert " ".join(f"{a}{m}" for a, m in sched(4, 1, 0)) == "F0 F1 dI0 dW0 F2 dI1 dW1 F3 dI2 dW2 dI3 dW3"
    assert peak_live(sched(8, 3, 3)) == 7 and peak_live(full_backward(sched(8, 3, 3))) == 4


def _run_chunks(schedule, M, steps, shapes, T=64, H=4):
    """Two chunks, one oracle linear each, own pools, one flat gradient buffer."""
    P = peak_live_per_chunk(schedule)
    offs, total = inputs.grad_offsets([("l", K, N) for K, N in shapes])
    layers = [OracleLinear(T, K, N, H, 0, P[c], stage=0, unit=c) for c, (K, N) in enumerate(shapes)]
    buf = np.zeros(total, np.float32)
    outs = {}
    for step in range(steps):
        for c, (K, N) in enumerate(shapes):
            layers[c].set_weight(inputs.bits(inputs.weights("CH", step, c, N, K)))
        tapes = {}
        for a, m, c in schedule:
            K, N = shapes[c]
            L = layers[c]
            if a == "F":
                X = inputs.bits(inputs.activations("CH", step, 0, c, m, T, K))
                tapes[(m, c)], outs[(step, "Y", m, c)] = L.forward(m, L.e_W, X)
            elif a == "dI":
                dY = inputs.bits(inputs.upstream_grads("CH", step, 0, c, m, T, N))
                outs[(step, "dX", m, c)] = L.backward_dI(tapes[(m, c)], dY)
            else:
                L.backward_dW(tapes[(m, c)], buf, offs[c])
        outs[(step, "mg")] = buf.copy()
        for L in layers:
            L.optimizer_boundary(M)
    return outs, [L.state() for L in layers]


@pytest.mark.parametrize("gen", ["interleaved", "zb_v"])
def test_two_chunk_split_equals_full_backward_bitwise_in_the_oracle(gen):
    M = 4
    s = interleaved_1f1b(M, 2, 0, 2, defer=2) if gen == "interleaved" else zb_v(M, 2, 1)
    a, sa = _run_chunks(s, M, 2, [(64, 96), (96, 64)])
    b, sb = _run_chunks(full_backward_chunks(s), M, 2, [(64, 96), (96, 64)])
    assert a.keys() == b.keys()
    for k in a:
        assert np.array_equal(a[k].view(np.uint8), b[k].view(np.uint8)), k
    for x, y in zip(sa, sb):
        assert state_equal({**x, "slots": []}, {**y, "slots": []})
        assert x["classes"]["X"]["count"] == 2 * M
