"""CPU-only checks of the C-ABI: the library loads, exports everything the header declares, and the
host contract core (no CUDA context) agrees with the oracle's state machine, incl. the fault table."""
import os
import re
import subprocess
import sys

import numpy as np
import pytest
from hypothesis import given, settings, strategies as st

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="session")
def qe():
    from paper_2609_23536_b200 import build

    build.build()
    from paper_2609_23536_b200 import binding

    return binding


def test_library_exports_every_declared_symbol(qe):
    header = open(os.path.join(ROOT, "include", "qe.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(qe_[a-z0-9_A-Z]+)\s*\(", header))
    assert len(declared) >= 40
    for name in sorted(declared):
        assert hasattr(qe.lib, name), name
    assert declared == set(qe._SIGNATURES), declared ^ set(qe._SIGNATURES)
    assert qe.lib.qe_abi_version() == 1
    assert qe.lib.qe_status_name(-7) == b"QE_ERR_STALE_REF"


def test_struct_sizes_match_header(qe):
    import ctypes as C

    assert C.sizeof(qe.qe_tape) == 40
    assert C.sizeof(qe.qe_slot_view) == 40
    assert C.sizeof(qe.qe_contract_view) == 48 + 40 * 64
    assert C.sizeof(qe.qe_layer_config) == 40 + 8 + 32


def test_contract_runs_without_cuda_context():
    # Table 3's injections run in a process that initialises no CUDA context: run one in a child
    # with no visible device and check that nothing tried to create a context.
    code = (
        "import sys; sys.path.insert(0, %r)\n"
        "from paper_2609_23536_b200 import binding as qe\n"
        "c = qe.Contract(2)\n"
        "t = c.forward_commit(0)\n"
        "c.dI_commit(t)\n"
        "try:\n    c.dI_commit(t)\nexcept qe.QEError as e:\n    print(e.code)\n"
    ) % ROOT
    env = dict(os.environ, CUDA_VISIBLE_DEVICES="")
    out = subprocess.run([sys.executable, "-c", code], capture_output=True, text=True, env=env)
    assert out.returncode == 0, out.stderr
    assert out.stdout.strip() == "DUP_CONSUME"


def _expect(qe, code, fn, *a):
    with pytest.raises(qe.QEError) as e:
        fn(*a)
    assert e.value.code == code, (e.value.code, code)


BUF, ELEMS, SLICE = 0x7F0000000000, 4096, 1024


def _full(c, mb):
    t = c.forward_commit(mb)
    c.dI_commit(t)
    c.dW_check(t, BUF, ELEMS, 0, SLICE)
    c.dW_commit(t, BUF, 0, SLICE)
    return t


def test_fault_table(qe):
    # 1 old reference after slot reuse: rejected at lookup, current record preserved
    c = qe.Contract(2)
    old = _full(c, 0)
    new = c.forward_commit(1)
    assert new.ref.slot == old.ref.slot and new.ref.gen == old.ref.gen + 1
    before = c.get()
    _expect(qe, "STALE_REF", c.dI_check, old)
    _expect(qe, "STALE_REF", c.dW_check, old, BUF, ELEMS, 0, SLICE)
    assert c.get() == before
    c.dI_commit(new)
    # 2 repeated dI
    _expect(qe, "DUP_CONSUME", c.dI_commit, new)
    # 3 finalize with one missing dW
    _expect(qe, "PENDING", c.boundary, 2)
    c.dW_commit(new, BUF, 0, SLICE)
    c2 = qe.Contract(2)
    _full(c2, 0)
    _expect(qe, "INCOMPLETE", c2.boundary, 2)
    assert c2.get()["e_W"] == 0
    # 4 write after an aborted write
    c3 = qe.Contract(2)
    t = c3.forward_commit(0)
    c3.dI_commit(t)
    c3.abort()
    _expect(qe, "ABORTED", c3.dW_check, t, BUF, ELEMS, 0, SLICE)
    _expect(qe, "ABORTED", c3.boundary, 1)
    c3.rebuild()
    _expect(qe, "STALE_REF", c3.dI_check, t)
    assert c3.forward_commit(0).ref.gen == 2
    # 5 stale weight cache
    c4 = qe.Contract(2)
    c4.forward_commit(0)
    c4.invalidate_cache()
    _expect(qe, "STALE_CACHE", c4.forward_check, 1, 0)
    # 6/7 checkpoint with a live tape
    c5 = qe.Contract(2)
    c5.checkpoint_check()
    t = c5.forward_commit(0)
    _expect(qe, "PENDING", c5.checkpoint_check)


def test_boundary_check_is_the_boundary_without_its_effects(qe):
    # the check half of the optimizer commit (Algorithm 1: a check precedes its action and changes nothing): the same
    # verdicts as the boundary itself, state untouched, so that several layers can be checked before any is committed
    c = qe.Contract(2)
    t = c.forward_commit(0)
    for code in ("PENDING",):
        before = c.get()
        _expect(qe, code, c.boundary_check, 1)
        assert c.get() == before
    c.dI_commit(t)
    c.dW_check(t, BUF, ELEMS, 0, SLICE)
    c.dW_commit(t, BUF, 0, SLICE)
    before = c.get()
    _expect(qe, "INCOMPLETE", c.boundary_check, 2)
    _expect(qe, "BAD_ARG", c.boundary_check, 0)
    c.boundary_check(1)
    c.boundary_check(1)  # as often as one likes
    assert c.get() == before and before["e_W"] == 0
    c.boundary(1)
    assert c.get()["e_W"] == 1 and c.get()["write_mask"] == 0
    c.abort()
    _expect(qe, "ABORTED", c.boundary_check, 1)


def test_destination_rules(qe):
    reg = qe.Registry()
    a, b = qe.Contract(1, unit=0, registry=reg), qe.Contract(1, unit=1, registry=reg)
    ta, tb = a.forward_commit(0), b.forward_commit(0)
    _expect(qe, "ORDER", a.dW_check, ta, BUF, ELEMS, 0, SLICE)
    a.dI_commit(ta)
    b.dI_commit(tb)
    _expect(qe, "DEST", a.dW_check, ta, 0, ELEMS, 0, SLICE)
    _expect(qe, "DEST", a.dW_check, ta, BUF, ELEMS, 2, SLICE)  # misaligned
    _expect(qe, "DEST", a.dW_check, ta, BUF, SLICE - 1, 0, SLICE)  # too small
    _expect(qe, "DEST", a.dW_check, ta, BUF, ELEMS, ELEMS, SLICE)
    assert a.dW_check(ta, BUF, ELEMS, 0, SLICE) is False  # first write overwrites
    a.dW_commit(ta, BUF, 0, SLICE)
    _expect(qe, "DEST", b.dW_check, tb, BUF, ELEMS, 512, SLICE)  # aliases a's slice
    b.dW_check(tb, BUF, ELEMS, 1024, SLICE)
    b.dW_commit(tb, BUF, 1024, SLICE)
    a.boundary(1)
    # bound destination is per epoch: after the boundary another one may be bound, but not b's
    t = a.forward_commit(0)
    a.dI_commit(t)
    _expect(qe, "DEST", a.dW_check, t, BUF, ELEMS, 1024, SLICE)
    a.dW_check(t, BUF, ELEMS, 2048, SLICE)


@settings(max_examples=80, deadline=None)
@given(st.lists(st.tuples(st.sampled_from(["F", "dI", "dW", "stale", "boundary", "abort"]), st.integers(0, 4)), max_size=50))
def test_contract_core_matches_oracle_state_machine(qe, ops):
    from oracle.layer import ContractError, OracleLinear, Tape, TapeKey, TapeRef
    from paper_2609_23536_b200 import inputs

    T = K = N = 16
    P = 3
    O = OracleLinear(T, K, N, 4, 0, P)
    O.set_weight(inputs.bits(inputs.weights("F", 0, 0, N, K)))
    X = inputs.bits(inputs.activations("F", 0, 0, 0, 0, T, K))
    dY = inputs.bits(inputs.upstream_grads("F", 0, 0, 0, 0, T, N))
    buf = np.zeros(N * K, np.float32)
    Cc = qe.Contract(P)
    tapes = []

    def both(ofn, cfn):
        oc = cc = None
        try:
            r = ofn()
        except ContractError as e:
            oc, r = e.code, None
        try:
            c = cfn()
        except qe.QEError as e:
            cc, c = e.code, None
        assert oc == cc, (oc, cc)
        return r, c

    def to_c(t):
        ct = qe.qe_tape()
        ct.key.epoch, ct.key.stage, ct.key.mb, ct.key.unit, ct.key.inv = t.key
        ct.ref.slot, ct.ref.gen = t.ref
        return ct

    for op, m in ops:
        if op == "F":
            r, c = both(lambda: O.forward(m, O.e_W, X), lambda: (Cc.forward_check(m, Cc.get()["e_W"]), Cc.forward_commit(m))[1])
            if r is not None:
                assert c.astuple() == (tuple(r[0].key), tuple(r[0].ref))
                tapes.append(r[0])
        elif op in ("dI", "stale") and tapes:
            t = tapes[m % len(tapes)]
            both(lambda: O.backward_dI(t, dY), lambda: Cc.dI_commit(to_c(t)))
        elif op == "dW" and tapes:
            t = tapes[m % len(tapes)]
            addr = buf.ctypes.data

            def cdw():
                Cc.dW_check(to_c(t), addr, buf.size, 0, N * K)
                Cc.dW_commit(to_c(t), addr, 0, N * K)

            both(lambda: O.backward_dW(t, buf, 0), cdw)
        elif op == "boundary":
            both(lambda: O.optimizer_boundary(m + 1), lambda: Cc.boundary(m + 1))
        elif op == "abort" and m == 0:
            O.abort_step()
            Cc.abort()
            both(lambda: O.arena_rebuild(), lambda: Cc.rebuild())
        so, sc = O.state(), Cc.get()
        for k in ("e_W", "e_C", "token", "write_mask", "fwd_in_epoch", "aborted", "slots"):
            assert so[k] == sc[k], (k, so[k], sc[k])


def test_contract_restore_is_the_restart_rule(qe):
    c = qe.Contract(2)
    t = c.forward_commit(0)
    _expect(qe, "PENDING", c.restore, 5)
    c.dI_commit(t)
    c.dW_check(t, BUF, ELEMS, 0, SLICE)
    c.dW_commit(t, BUF, 0, SLICE)
    c.restore(5)
    v = c.get()
    assert v["e_W"] == 5 and v["e_C"] == qe.QE_INVALID_EPOCH and v["write_mask"] == 0 and v["fwd_in_epoch"] == 0
    assert v["token"] == 2 and v["slots"][0]["gen"] == 1  # process-local identities keep counting
    refresh, slot = c.forward_check(0, 5)
    assert refresh and slot == 0
    _expect(qe, "EPOCH", c.forward_check, 0, 0)
