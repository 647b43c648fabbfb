"""Pins for the oracle's F / dI / dW state machine (CPU only): invariants of the contract."""
from fractions import Fraction

import numpy as np
import pytest
from hypothesis import given, settings, strategies as st

from harness import c1_inputs, run_oracle_steps, state_equal
from oracle import bf16, fp8
from oracle.layer import ArenaRegistry, ContractError, OracleLinear, Tape, TapeKey, TapeRef
from oracle.scaling import amax_bf16
from paper_2609_23536_b200 import inputs
from paper_2609_23536_b200.schedules import full_backward, peak_live, sched


def _weights(T=64, K=64, N=64, cfg="C1s"):
    w0 = inputs.weights(cfg, 0, 0, N, K)
    ws = [w0]
    for e in range(1, 8):
        ws.append(inputs.optimizer_perturbation(ws[-1], cfg, e, 0, 0))
    return [inputs.bits(w) for w in ws]


def _small(T=64, K=64, N=96, H=4, P=4):
    return OracleLinear(T, K, N, H, 0, P)


def _get_inputs(T, K, N):
    return lambda step, mb: c1_inputs(step, mb, T, K, N, cfg="C1s")


def test_split_equals_full_backward_bitwise_across_rollover():
    # Paper Sec. 5.2 (state checks): split F/dI/dW against full backward, exact, across the
    # four-entry amax-history rollover.
    T, K, N, M = 64, 64, 96, 4
    W = _weights(T, K, N)
    s = sched(M, 2, 1)
    runs = []
    for schedule in (s, full_backward(s)):
        L = _small(T, K, N, H=4, P=peak_live(s))
        buf = np.zeros(N * K + 8, np.float32)
        runs.append((run_oracle_steps(L, schedule, 3, M, buf, 4, _get_inputs(T, K, N), lambda e: W[e]), L.state()))
    (a, sa), (b, sb) = runs
    assert a.keys() == b.keys()
    for k in a:
        assert np.array_equal(a[k].view(np.uint8), b[k].view(np.uint8)), k
    # slot generations are process-local identities and depend on the reuse pattern; all else is equal
    assert state_equal({**sa, "slots": []}, {**sb, "slots": []})
    assert sa["classes"]["X"]["count"] == 12 > 4  # rolled over
    assert sa["classes"]["W"]["count"] == 3


def test_dW_never_touches_scale_state_and_token_counts_F_plus_dI():
    T, K, N, M = 64, 64, 96, 4
    W = _weights(T, K, N)
    L = _small(T, K, N)
    buf = np.zeros(N * K, np.float32)
    seen = {"F": 0, "dI": 0}
    last = {}

    def on_action(step, a, m, layer):
        st_ = layer.state()
        if a == "dW":
            assert state_equal({**st_, "write_mask": 0, "slots": []}, {**last["s"], "write_mask": 0, "slots": []})
        else:
            seen[a] += 1
        assert st_["token"] == seen["F"] + seen["dI"]
        last["s"] = st_

    run_oracle_steps(L, sched(M, 1, 0), 2, M, buf, 0, _get_inputs(T, K, N), lambda e: W[e], on_action)
    assert L.token == 2 * 2 * M


def test_delayed_scale_and_tape_snapshots():
    # the scale used at F(m) is the one committed before it; dW uses the snapshots in the tape
    T, K, N = 64, 64, 96
    W = _weights(T, K, N)
    L = _small(T, K, N)
    L.set_weight(W[0])
    X0, dY0 = c1_inputs(0, 0, T, K, N, "C1s")
    X1, dY1 = c1_inputs(0, 1, T, K, N, "C1s")
    t0, Y0 = L.forward(0, 0, X0)
    # first action: scale 1 everywhere -> Xq is the plain cast of X
    assert np.array_equal(L.slots[0].Xq, fp8.encode(bf16.decode(X0), fp8.E4M3))
    aX0 = amax_bf16(bf16.decode(X0))
    assert L.S["X"].scale == np.float32(np.float32(448.0) / aX0)
    t1, _ = L.forward(1, 0, X1)
    assert L.slots[1].sinv_X == np.float32(np.float32(1.0) / np.float32(np.float32(448.0) / aX0))
    assert L.slots[0].sinv_X == np.float32(1.0)
    L.backward_dI(t0, dY0)
    L.backward_dI(t1, dY1)
    sG0, sG1 = L.slots[0].sinv_G, L.slots[1].sinv_G
    assert sG0 == 1.0 and sG1 != 1.0
    buf = np.zeros(N * K, np.float32)
    L.backward_dW(t0, buf, 0)
    G = fp8.decode(fp8.encode(bf16.decode(dY0), fp8.E5M2), fp8.E5M2)
    Xd = fp8.decode(fp8.encode(bf16.decode(X0), fp8.E4M3), fp8.E4M3)
    assert np.array_equal(buf.reshape(N, K), (G.T @ Xd).astype(np.float32))


def test_weight_cache_refreshed_once_per_epoch():
    T, K, N = 64, 64, 96
    W = _weights(T, K, N)
    L = _small(T, K, N)
    L.set_weight(W[0])
    X0, dY0 = c1_inputs(0, 0, T, K, N, "C1s")
    t0, _ = L.forward(0, 0, X0)
    Wq0 = L.Wq.copy()
    assert L.e_C == 0 and L.S["W"].count == 1
    L.set_weight(W[1])  # parameters changed without a boundary: cache must NOT follow
    t1, _ = L.forward(1, 0, X0)
    assert np.array_equal(L.Wq, Wq0) and L.S["W"].count == 1
    buf = np.zeros(N * K, np.float32)
    for t in (t0, t1):
        L.backward_dI(t, dY0)
        L.backward_dW(t, buf, 0)
    L.optimizer_boundary(2)
    assert L.e_W == 1 and L.e_C == 0
    L.forward(0, 1, X0)
    assert L.e_C == 1 and L.S["W"].count == 2 and not np.array_equal(L.Wq, Wq0)


# ---------------------------------------------------------------- fault injections (Table 3)
def _primed(M=2, P=2):
    T, K, N = 32, 32, 32
    L = OracleLinear(T, K, N, 4, 0, P)
    L.set_weight(inputs.bits(inputs.weights("F", 0, 0, N, K)))
    X, dY = c1_inputs(0, 0, T, K, N, "F")
    buf = np.zeros(N * K, np.float32)
    return L, X, dY, buf


def _expect(code, fn, *a):
    with pytest.raises(ContractError) as e:
        fn(*a)
    assert e.value.code == code
    return e.value


def test_fault_old_reference_after_slot_reuse_preserves_current_record():
    L, X, dY, buf = _primed()
    t_old, _ = L.forward(0, 0, X)
    L.backward_dI(t_old, dY)
    L.backward_dW(t_old, buf, 0)
    t_new, _ = L.forward(1, 0, X)
    assert t_new.ref.slot == t_old.ref.slot and t_new.ref.gen == t_old.ref.gen + 1
    before = L.state()
    _expect("STALE_REF", L.backward_dI, t_old, dY)
    _expect("STALE_REF", L.backward_dW, t_old, buf, 0)
    assert state_equal(before, L.state())
    L.backward_dI(t_new, dY)  # current record still usable


def test_fault_repeated_dI_consumption():
    L, X, dY, buf = _primed()
    t, _ = L.forward(0, 0, X)
    L.backward_dI(t, dY)
    before = L.state()
    _expect("DUP_CONSUME", L.backward_dI, t, dY)
    assert state_equal(before, L.state())


def test_fault_finalize_with_missing_dW():
    L, X, dY, buf = _primed()
    t0, _ = L.forward(0, 0, X)
    t1, _ = L.forward(1, 0, X)
    L.backward_dI(t0, dY)
    L.backward_dW(t0, buf, 0)
    L.backward_dI(t1, dY)
    _expect("PENDING", L.optimizer_boundary, 2)  # live tape still holds the missing dW
    assert L.e_W == 0
    # and with the tape gone but the write missing: incomplete
    L2, X, dY, buf = _primed()
    t0, _ = L2.forward(0, 0, X)
    L2.backward_dI(t0, dY)
    L2.backward_dW(t0, buf, 0)
    _expect("INCOMPLETE", L2.optimizer_boundary, 2)
    assert L2.e_W == 0 and L2.write_mask == 1


def test_fault_write_after_aborted_write_requires_rebuild():
    L, X, dY, buf = _primed()
    t0, _ = L.forward(0, 0, X)
    L.backward_dI(t0, dY)
    L.abort_step()
    assert L.live_tapes() == 0 and L.slots[0].gen == 1
    _expect("ABORTED", L.backward_dW, t0, buf, 0)
    _expect("ABORTED", L.forward, 0, 0, X)
    _expect("ABORTED", L.optimizer_boundary, 2)
    L.arena_rebuild()
    t, _ = L.forward(0, 0, X)
    assert t.ref == TapeRef(0, 2)
    _expect("STALE_REF", L.backward_dI, t0, dY)


def test_fault_stale_weight_cache():
    L, X, dY, buf = _primed()
    L.forward(0, 0, X)
    L.invalidate_cache()
    before = L.state()
    _expect("STALE_CACHE", L.forward, 1, 0, X)
    assert state_equal(before, L.state())


def test_fault_checkpoint_with_live_tape_is_withheld():
    L, X, dY, buf = _primed()
    L.checkpoint_allowed()
    t, _ = L.forward(0, 0, X)
    _expect("PENDING", L.checkpoint_allowed)
    L.backward_dI(t, dY)
    _expect("PENDING", L.checkpoint_allowed)
    L.backward_dW(t, buf, 0)
    L.checkpoint_allowed()


def test_other_rejections():
    L, X, dY, buf = _primed(P=2)
    t0, _ = L.forward(0, 0, X)
    _expect("KEY_LIVE", L.forward, 0, 0, X)
    _expect("EPOCH", L.forward, 1, 5, X)
    _expect("ORDER", L.backward_dW, t0, buf, 0)  # dW before dI
    t1, _ = L.forward(1, 0, X)
    _expect("POOL_FULL", L.forward, 2, 0, X)
    _expect("KEY_MISMATCH", L.backward_dI, Tape(TapeKey(0, 0, 1, 0, 0), t0.ref), dY)
    L.backward_dI(t1, dY)
    _expect("ORDER", L.backward_dW, t1, buf, 0)  # first write of the epoch must be microbatch 0
    L.backward_dI(t0, dY)
    _expect("DEST", L.backward_dW, t0, buf, 2)  # misaligned
    _expect("DEST", L.backward_dW, t0, buf[: 32 * 32 - 1], 0)  # too small
    L.backward_dW(t0, buf, 0)
    _expect("DEST", L.backward_dW, t1, np.zeros_like(buf), 0)  # not the bound destination
    L.backward_dW(t1, buf, 0)
    # a second tape for microbatch 0 in the same epoch: its write is a duplicate
    t0b, _ = L.forward(0, 0, X)
    L.backward_dI(t0b, dY)
    _expect("DUP_WRITE", L.backward_dW, t0b, buf, 0)


def test_aliased_destinations_across_layers_fail():
    reg = ArenaRegistry()
    A = OracleLinear(32, 32, 32, 4, 0, 1, registry=reg)
    B = OracleLinear(32, 32, 32, 4, 0, 1, unit=1, registry=reg)
    w = inputs.bits(inputs.weights("F", 0, 0, 32, 32))
    X, dY = c1_inputs(0, 0, 32, 32, 32, "F")
    buf = np.zeros(3 * 1024, np.float32)
    for L in (A, B):
        L.set_weight(w)
    ta, _ = A.forward(0, 0, X)
    tb, _ = B.forward(0, 0, X)
    A.backward_dI(ta, dY)
    B.backward_dI(tb, dY)
    A.backward_dW(ta, buf, 0)
    _expect("DEST", B.backward_dW, tb, buf, 512)
    B.backward_dW(tb, buf, 1024)


# ---------------------------------------------------------------- pool vs dict model
@settings(max_examples=60, deadline=None)
@given(st.lists(st.tuples(st.sampled_from(["F", "dI", "dW", "stale"]), st.integers(0, 5)), max_size=40))
def test_pool_against_dict_model(ops):
    T = K = N = 32
    P = 3
    L = OracleLinear(T, K, N, 4, 0, P)
    L.set_weight(inputs.bits(inputs.weights("F", 0, 0, N, K)))
    X, dY = c1_inputs(0, 0, T, K, N, "F")
    buf = np.zeros(N * K, np.float32)
    live, gens, released, written = {}, [0] * P, [], set()
    for op, m in ops:
        if op == "F":
            free = [p for p in range(P) if p not in [t.ref.slot for t, _ in live.values()]]
            if m in live:
                _expect("KEY_LIVE", L.forward, m, 0, X)
            elif not free:
                _expect("POOL_FULL", L.forward, m, 0, X)
            else:
                t, _ = L.forward(m, 0, X)
                gens[free[0]] += 1
                assert t.ref == TapeRef(free[0], gens[free[0]])  # lowest free slot, generation +1
                live[m] = (t, 0)
        elif op == "dI" and m in live:
            t, bits = live[m]
            if bits & 1:
                _expect("DUP_CONSUME", L.backward_dI, t, dY)
            else:
                L.backward_dI(t, dY)
                live[m] = (t, bits | 1)
        elif op == "dW" and m in live:
            t, bits = live[m]
            if not bits & 1:
                _expect("ORDER", L.backward_dW, t, buf, 0)
            elif m in written:
                _expect("DUP_WRITE", L.backward_dW, t, buf, 0)
            elif not written and m != 0:
                _expect("ORDER", L.backward_dW, t, buf, 0)
            else:
                L.backward_dW(t, buf, 0)
                written.add(m)
                released.append(t)
                del live[m]
        elif op == "stale" and released:
            _expect("STALE_REF", L.backward_dI, released[m % len(released)], dY)
        assert L.live_tapes() == len(live)
        assert [s.gen for s in L.slots] == gens
        assert len({t.ref.slot for t, _ in live.values()}) == len(live)  # injective


def test_resume_from_quiescent_checkpoint_equals_uninterrupted_run():
    # Sec. 5.2: save at step 3, continue through step 8, compare with the uninterrupted run.  Persistent state
    # (histories, scales, weight version) is restored; tokens and generations are process-local; the cache refreshes.
    T, K, N, M, H = 64, 64, 96, 4, 4
    W = _weights(T, K, N)
    s = sched(M, 2, 1)
    get = _get_inputs(T, K, N)

    def run(L, buf, steps):
        outs = {}
        for step in steps:
            L.set_weight(W[step])
            tapes = {}
            for a, m in s:
                X, dY = get(step, m)
                if a == "F":
                    tapes[m], outs[(step, "Y", m)] = L.forward(m, L.e_W, X)
                elif a == "dI":
                    outs[(step, "dX", m)] = L.backward_dI(tapes[m], dY)
                else:
                    L.backward_dW(tapes[m], buf, 0)
            outs[(step, "mg")] = buf.copy()
            L.optimizer_boundary(M)
        return outs

    A = _small(T, K, N, H=H, P=peak_live(s))
    bufA = np.zeros(N * K, np.float32)
    full = run(A, bufA, range(8))

    B = _small(T, K, N, H=H, P=peak_live(s))
    bufB = np.zeros(N * K, np.float32)
    run(B, bufB, range(3))
    B.set_weight(W[3])
    t, _ = B.forward(0, B.e_W, get(3, 0)[0])
    _expect("PENDING", B.save_state)  # checkpoint withheld while a tape is live
    B.backward_dI(t, get(3, 0)[1])
    B.backward_dW(t, bufB, 0)
    B.abort_step()
    B.arena_rebuild()
    saved = B.save_state()

    C = _small(T, K, N, H=H, P=peak_live(s))  # the "fresh process"
    C.load_state(saved)
    assert C.e_W == 3 and C.e_C != 3 and C.token == 0
    bufC = np.zeros(N * K, np.float32)
    # the interrupted process had already run (and abandoned) one microbatch of step 3: its X/G/Y commits are part of
    # the saved state, so the resumed suffix is compared with an uninterrupted run that did the same
    A2 = _small(T, K, N, H=H, P=peak_live(s))
    buf2 = np.zeros(N * K, np.float32)
    run(A2, buf2, range(3))
    A2.set_weight(W[3])
    t, _ = A2.forward(0, A2.e_W, get(3, 0)[0])
    A2.backward_dI(t, get(3, 0)[1])
    A2.backward_dW(t, buf2, 0)
    A2.abort_step()
    A2.arena_rebuild()
    want = run(A2, buf2, range(3, 8))
    got = run(C, bufC, range(3, 8))
    for k in want:
        assert np.array_equal(want[k].view(np.uint8), got[k].view(np.uint8)), k
    sa, sc = A2.state(), C.state()
    assert state_equal({**sa, "slots": [], "token": 0}, {**sc, "slots": [], "token": 0})
    assert sa["token"] != sc["token"]  # process-local
    # and a clean save at a step boundary resumes onto the plain uninterrupted trajectory
    D = _small(T, K, N, H=H, P=peak_live(s))
    bufD = np.zeros(N * K, np.float32)
    run(D, bufD, range(3))
    E = _small(T, K, N, H=H, P=peak_live(s))
    E.load_state(D.save_state())
    bufE = np.zeros(N * K, np.float32)
    got = run(E, bufE, range(3, 8))
    for k in got:
        assert np.array_equal(full[k].view(np.uint8), got[k].view(np.uint8)), k


# ------------------------------------------------------------------------------------------ per-microbatch arena
def _int_layer_run(M, T, K, N, use_arena, seed=5):
    """Integer-valued X (|x| <= 7) and dY (|g| <= 7), each containing a 7: every scale is a power of two (448/7,
    57344/7) and every per-microbatch gradient sum_t g x is a small integer, exact in bf16 and FP32."""
    rng = np.random.default_rng(seed)
    L = OracleLinear(T, K, N, 4, 0, M)
    L.set_weight(inputs.bits(inputs.weights("AR", 0, 0, N, K)))
    n = N * K
    arena = np.full(16 + M * n, 0x7FC0, np.uint16)  # NaN-filled: an unwritten view would show
    buf = np.full(8 + n, np.float32(99.0))
    exact = np.zeros((N, K), np.int64)
    tapes = []
    for m in range(M):
        x = rng.integers(-7, 8, (T, K))
        g = rng.integers(-7, 8, (T, N))
        x[0, 0], g[0, 0] = 7, -7
        exact += g.T @ x
        import torch

        tape, _ = L.forward(m, L.e_W, inputs.bits(torch.tensor(x, dtype=torch.float32).to(torch.bfloat16)))
        L.backward_dI(tape, inputs.bits(torch.tensor(g, dtype=torch.float32).to(torch.bfloat16)))
        tapes.append(tape)
    for m in range(M):
        if use_arena:
            L.backward_dW_arena(tapes[m], arena, 16, M)
        else:
            L.backward_dW(tapes[m], buf, 8)
    if use_arena:
        L.arena_finalize(arena, 16, M, buf, 8)
    return L, arena, buf, exact


def test_arena_variant_equals_flat_accumulate_and_integer_matmul_when_views_are_exact():
    M, T, K, N = 4, 4, 8, 16
    La, arena, buf_a, exact = _int_layer_run(M, T, K, N, True)
    Lf, _, buf_f, exact_f = _int_layer_run(M, T, K, N, False)
    assert np.array_equal(exact, exact_f) and np.abs(exact).max() < 2**24
    assert np.array_equal(buf_a[8:].reshape(N, K), exact.astype(np.float32))
    assert np.array_equal(buf_a.view(np.uint32), buf_f.view(np.uint32))
    assert np.all(buf_a[:8] == 99.0)  # nothing outside the slice
    assert np.all(arena[:16] == 0x7FC0)
    views = bf16.decode(arena[16:]).reshape(M, N, K)
    assert np.array_equal(views.sum(axis=0), exact.astype(np.float64))  # every view holds its own microbatch
    assert not np.array_equal(views[0], views[1])
    assert state_equal(La.state(), Lf.state())
    La.optimizer_boundary(M)


def _nearest_bf16_by_search(x: Fraction) -> int:
    """Nearest bf16 code to an exact rational, ties to the even code, by searching all finite codes."""
    best, best_err = None, None
    for code in range(0x10000):
        if (code & 0x7F80) == 0x7F80:
            continue
        v = Fraction(float(bf16.decode(np.array([code], np.uint16))[0]))
        err = abs(v - x)
        if best is None or err < best_err or (err == best_err and code % 2 == 0 and best % 2 == 1):
            best, best_err = code, err
    return best


def test_arena_view_is_one_rounding_of_the_exact_gradient_to_bf16():
    T, K, N = 3, 2, 2
    L = OracleLinear(T, K, N, 4, 0, 1)
    L.set_weight(inputs.bits(inputs.weights("AR", 0, 0, N, K)))
    X = inputs.bits(inputs.activations("AR", 0, 0, 0, 0, T, K))
    dY = inputs.bits(inputs.upstream_grads("AR", 0, 0, 0, 0, T, N))
    L.S["X"].scale, L.S["X"].scale_inv = np.float32(3.7), np.float32(1.0) / np.float32(3.7)
    L.S["G"].scale, L.S["G"].scale_inv = np.float32(811.0), np.float32(1.0) / np.float32(811.0)
    tape, _ = L.forward(0, L.e_W, X)
    L.backward_dI(tape, dY)
    s = L.slots[tape.ref.slot]
    Gd, Xd = fp8.decode(s.Gq, fp8.E5M2), fp8.decode(s.Xq, fp8.E4M3)
    sg, sx = Fraction(float(s.sinv_G)), Fraction(float(s.sinv_X))
    arena = np.zeros(8, np.uint16)
    L.backward_dW_arena(tape, arena, 0, 1)
    for n in range(N):
        for k in range(K):
            exact = sum(Fraction(float(Gd[t, n])) * Fraction(float(Xd[t, k])) for t in range(T)) * sg * sx
            assert int(arena[n * K + k]) == _nearest_bf16_by_search(exact), (n, k)


def test_arena_finalize_adds_views_in_microbatch_order_in_fp32():
    L = OracleLinear(1, 1, 8, 4, 0, 3)
    L.write_mask, n = 0b111, 8
    one, tiny = 0x3F80, 0x3380  # bf16 1.0 and 2^-24
    assert bf16.decode(np.array([tiny], np.uint16))[0] == 2.0**-24
    buf = np.zeros(8, np.float32)
    for order, want in (((one, tiny, tiny), np.float32(1.0)), ((tiny, tiny, one), np.float32(1.0) + np.float32(2.0**-23))):
        arena = np.concatenate([np.full(n, c, np.uint16) for c in order])
        L.bound_dest = (id(arena), 0)
        L.arena_finalize(arena, 0, 3, buf, 0)
        assert np.all(buf == want) and want.dtype == np.float32


def test_arena_contract_errors():
    M, T, K, N = 2, 4, 8, 8
    L, arena, buf, _ = _int_layer_run(M, T, K, N, True)
    with pytest.raises(ContractError) as e:
        L.arena_finalize(arena, 24, M, buf, 8)  # not the bound region
    assert e.value.code == "DEST"
    L.optimizer_boundary(M)
    # next epoch: one view missing -> finalize refuses; duplicate write refused; region too small refused
    import torch

    L.set_weight(inputs.bits(inputs.weights("AR", 1, 0, N, K)))
    x = inputs.bits(torch.ones((T, K), dtype=torch.bfloat16))
    g = inputs.bits(torch.ones((T, N), dtype=torch.bfloat16))
    t0, _ = L.forward(0, L.e_W, x)
    t1, _ = L.forward(1, L.e_W, x)
    L.backward_dI(t0, g)
    L.backward_dI(t1, g)
    with pytest.raises(ContractError) as e:
        L.backward_dW_arena(t1, arena, 16, M)
    assert e.value.code == "ORDER"  # microbatch 0 first
    with pytest.raises(ContractError) as e:
        L.backward_dW_arena(t0, arena[: 16 + N * K], 16, M)
    assert e.value.code == "DEST"
    L.backward_dW_arena(t0, arena, 16, M)
    with pytest.raises(ContractError) as e:
        L.arena_finalize(arena, 16, M, buf, 8)
    assert e.value.code == "INCOMPLETE"
    with pytest.raises(ContractError) as e:
        L.backward_dW_arena(t0, arena, 16, M)
    assert e.value.code in ("STALE_REF", "DUP_CONSUME", "DUP_WRITE")
    L.backward_dW_arena(t1, arena, 16, M)
    L.arena_finalize(arena, 16, M, buf, 8)
    assert np.all(buf[8:] == 2 * T)
    L.optimizer_boundary(M)
