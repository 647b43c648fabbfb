"""GPU parity at the benchmark configurations' full sizes (configs 2-5), through the C-ABI.

State (amax windows, scales, inverse scales, token, versions, tapes, write masks) is compared with the
oracle bit for bit after EVERY action of every linear.  FP8 bytes and GEMM outputs are compared on a
sample of (step, linear, microbatch) units -- the oracle's float64 GEMMs and software casts over every
unit of these sizes would take hours -- with GEMM outputs checked on sampled rows computed one by one.
Within the GPU path, graph replay vs eager and staged vs direct placement are compared bitwise in full."""
import numpy as np
import pytest
import torch

from harness import (assert_gemm_close, assert_grad_close, dW_abs_products, state_equal, state_equal_except_Y,
                     transposed_or_none)
from oracle import bf16
from oracle.layer import ArenaRegistry, OracleLinear
from paper_2609_23536_b200 import inputs
from paper_2609_23536_b200.schedules import peak_live, sched

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module")
def qe():
    from paper_2609_23536_b200 import build

    build.build()
    from paper_2609_23536_b200 import binding

    return binding


class Stage:
    """The linears of a configuration on the GPU and, optionally, in the oracle, driven in lock step."""

    def __init__(self, qe, name, mode, with_oracle=True, n_layers=None, staged=False):
        cfg = inputs.CONFIGS[name]
        self.qe, self.name, self.cfg = qe, name, cfg
        self.T, self.M = cfg["T"], cfg["M"]
        self.schedule = sched(self.M, *cfg["sched"])
        self.P = peak_live(self.schedule)
        L = cfg["layers"] if n_layers is None else n_layers
        self.units = [(l, j, K, N) for l in range(L) for j, (_, K, N) in enumerate(cfg["linears"])]
        offs, per_layer = inputs.grad_offsets(cfg["linears"])
        self.offsets = [l * per_layer + offs[j] for l, j, _, _ in self.units]
        self.ctx = qe.Context(mode)
        self.grad = torch.full((per_layer * L,), 3.0, device=DEV)  # stale contents: mb 0 must overwrite
        self.temp = torch.empty(max(K * N for _, _, K, N in self.units), device=DEV) if staged else None
        self.W = [inputs.weights(name, l, j, N, K) for l, j, K, N in self.units]
        self.G = [qe.Layer(self.ctx, self.T, K, N, cfg["H"], cfg["margin"], self.P, self.W[u].to(DEV), unit=u)
                  for u, (l, j, K, N) in enumerate(self.units)]
        self.O = None
        if with_oracle:
            reg = ArenaRegistry()
            self.O = [OracleLinear(self.T, K, N, cfg["H"], cfg["margin"], self.P, unit=u, registry=reg)
                      for u, (l, j, K, N) in enumerate(self.units)]
            self.ograd = np.zeros(per_layer * L, np.float32)  # lazily committed: only sampled rows are touched
            self.oabs = {}  # unit -> sum over the heavy microbatches of sum_t |g x| alpha on the sampled gradient rows
        self.epoch = 0

    def x(self, step, u, mb):
        l, j, K, N = self.units[u]
        if self.name == "C4":
            return inputs.stress_activations(step, mb, self.T, K)
        return inputs.activations(self.name, step, l, j, mb, self.T, K)

    def dy(self, step, u, mb):
        l, j, K, N = self.units[u]
        return inputs.upstream_grads(self.name, step, l, j, mb, self.T, N)

    def run_step(self, step, heavy=lambda u, mb: False, rows=None, keep=None, check_state=True):
        """keep(u, mb, kind) -> True to retain the GPU output (as bits) in the returned dict."""
        outs, gt, ot = {}, {}, {}
        if step > 0:
            for u, (l, j, K, N) in enumerate(self.units):
                self.W[u] = inputs.optimizer_perturbation(self.W[u], self.name, step, l, j)
                self.G[u].weight.copy_(self.W[u].to(DEV))
        if self.O:
            for u in range(len(self.units)):
                self.O[u].set_weight(inputs.bits(self.W[u]))
        n = len(self.units)
        for a, m in self.schedule:
            for u in (range(n) if a == "F" else range(n - 1, -1, -1)):
                l, j, K, N = self.units[u]
                G, h = self.G[u], heavy(u, m)
                r = rows(u) if rows else None
                if a == "F":
                    xb = self.x(step, u, m)
                    y = torch.empty((self.T, N), dtype=torch.bfloat16, device=DEV)
                    gt[(u, m)] = G.forward(m, self.epoch, xb.to(DEV), y)
                    if keep and keep(u, m, "Y"):
                        outs[(u, m, "Y")] = inputs.bits(y.cpu())
                    if self.O:
                        ot[(u, m)], oy = self.O[u].forward(m, self.epoch, inputs.bits(xb), rows=r[0] if r else [0], light=not h)
                        assert gt[(u, m)].astuple() == (tuple(ot[(u, m)].key), tuple(ot[(u, m)].ref))
                        if h:
                            p = gt[(u, m)].ref.slot
                            assert np.array_equal(G.read_fp8(0, p), self.O[u].slots[p].Xq), ("Xq", step, u, m)
                            xt, wt = transposed_or_none(G, 1, p), transposed_or_none(G, 5)
                            assert xt is None or np.array_equal(xt, self.O[u].slots[p].Xq.T)
                            assert np.array_equal(G.read_fp8(4), self.O[u].Wq) and (wt is None or np.array_equal(wt, self.O[u].Wq.T))
                            assert_gemm_close(inputs.bits(y[r[0]].cpu()), oy, ("Y", step, u, m))
                elif a == "dI":
                    gb = self.dy(step, u, m)
                    dx = torch.empty((self.T, K), dtype=torch.bfloat16, device=DEV)
                    G.backward_dI(gt[(u, m)], gb.to(DEV), dx)
                    if keep and keep(u, m, "dX"):
                        outs[(u, m, "dX")] = inputs.bits(dx.cpu())
                    if self.O:
                        odx = self.O[u].backward_dI(ot[(u, m)], inputs.bits(gb), rows=r[0] if r else [0], light=not h)
                        if h:
                            p = gt[(u, m)].ref.slot
                            assert np.array_equal(G.read_fp8(2, p), self.O[u].slots[p].Gq), ("Gq", step, u, m)
                            gt_ = transposed_or_none(G, 3, p)
                            assert gt_ is None or np.array_equal(gt_, self.O[u].slots[p].Gq.T)
                            assert_gemm_close(inputs.bits(dx[r[0]].cpu()), odx, ("dX", step, u, m))
                else:
                    if self.temp is not None:
                        G.backward_dW_staged(gt[(u, m)], self.grad, self.offsets[u], self.temp)
                    else:
                        G.backward_dW(gt[(u, m)], self.grad, self.offsets[u])
                    if self.O:
                        slot = self.O[u].slots[ot[(u, m)].ref.slot]
                        if r and slot.Xq is not None and slot.Gq is not None:
                            if m == 0:
                                self.oabs.pop(u, None)
                            self.oabs[u] = self.oabs.get(u, 0.0) + dW_abs_products(slot, r[1])
                        self.O[u].backward_dW(ot[(u, m)], self.ograd, self.offsets[u], rows=r[1] if r else [0])
                if self.O and check_state:
                    g = G.state()
                    assert g["device_status"] == 0 and g["device_token"] == g["token"]
                    assert state_equal_except_Y(g, self.O[u].state()), (step, a, m, u)
        torch.cuda.synchronize()
        return outs

    def grads_match(self, u, rows_n, what):
        """main_grad rows of unit u against the oracle's accumulation (all microbatches heavy for u): Frobenius norm
        and every element within the FP32 accumulation bound."""
        l, j, K, N = self.units[u]
        got = self.grad[self.offsets[u]: self.offsets[u] + N * K].view(N, K)[rows_n].cpu().numpy()
        want = self.ograd[self.offsets[u]: self.offsets[u] + N * K].reshape(N, K)[rows_n]
        assert_grad_close(got, want, (what, u), abs_products=self.oabs[u], rel_tol=1e-5, contraction=self.T)

    def boundary(self):
        for G in self.G:
            G.optimizer_boundary(self.M)
        if self.O:
            for O in self.O:
                O.optimizer_boundary(self.M)
        self.epoch += 1


def _rows(T, N, nr, seed):
    rng = np.random.default_rng(seed)
    return (sorted(rng.choice(T, nr, replace=False).tolist() + [0, T - 1]),
            sorted(rng.choice(N, nr, replace=False).tolist() + [0, N - 1]))


def _tile_rows(T, N, seed):
    """One row in every 128-row tile of the token dimension (rows of Y / dX) and of the out-feature dimension (rows of
    the gradient slice), plus the first and last row: every output tile of every GEMM, both CTAs of a pair and every
    wave of the tile walk are then compared with the oracle somewhere."""
    pick = lambda n, mul: sorted({0, n - 1} | {128 * i + (mul * i + seed) % 128 for i in range(n // 128)})
    return pick(T, 37), pick(N, 53)


def test_config2_llama_block_state_every_action_bytes_and_gemm_rows_sampled(qe):
    # 4 linears, T = 2048, H = 1024, 8 microbatches in zero-bubble order, one flat gradient buffer.
    S = Stage(qe, "C2", qe.GRAPH)
    # one token row per 128-row tile of Y / dX and one gradient row per 128-row tile of every slice; every microbatch
    # heavy, so that all four gradient slices (the 92 MB gate/up one included) can be checked element by element
    rows = lambda u: _tile_rows(S.T, S.units[u][3], u)
    S.run_step(0, lambda u, m: True, rows)
    for u in range(4):
        S.grads_match(u, rows(u)[1], "C2")
    S.boundary()
    st = S.ctx.stats()
    assert st["graphs_built"] == len(S.units) * (3 * S.P + 1)
    assert st["kernels_launched"] == len(S.units) * (S.M * 5 + 1)


def test_config2_graph_replay_equals_eager_bitwise_in_full(qe):
    res = []
    for mode in (qe.EAGER, qe.GRAPH):
        S = Stage(qe, "C2", mode, with_oracle=False)
        outs = {}
        for step in range(2):
            o = S.run_step(step, keep=lambda u, m, k: m in (0, 7))
            outs.update({(step,) + k: v for k, v in o.items()})
            outs[(step, "mg")] = S.grad.cpu().numpy().copy()
            S.boundary()
        res.append((outs, [G.state() for G in S.G]))
    (a, sa), (b, sb) = res
    assert a.keys() == b.keys()
    for k in a:
        assert np.array_equal(a[k].view(np.uint8), b[k].view(np.uint8)), k
    for x, y in zip(sa, sb):
        for c in "XWGY":
            assert np.array_equal(x["classes"][c]["window"].view(np.uint32), y["classes"][c]["window"].view(np.uint32))
            assert x["classes"][c]["scale"].view(np.uint32) == y["classes"][c]["scale"].view(np.uint32)
        assert x["device_token"] == y["device_token"] == 2 * 2 * 8


def test_config4_scale_rollover_stress_step_by_step(qe):
    # Student-t activations, x1000 spike on 0.1 % of elements at step 5, x1e-3 collapse at step 9; H = 16,
    # margin 1, dW deferred by up to 6 schedule slots.  State after every action; bytes and GEMM rows on mb 0 of
    # every step and on every microbatch of the spike step (whose gradient slice is then checked too).
    S = Stage(qe, "C4", qe.GRAPH)
    rows = lambda u: _rows(S.T, 4096, 6, 4)
    scales = []
    for step in range(12):
        S.run_step(step, (lambda u, m: True) if step == 5 else (lambda u, m: m == 0), rows)
        if step == 5:
            S.grads_match(0, rows(0)[1], "C4 spike step")
        S.boundary()
        scales.append(float(S.G[0].state()["classes"]["X"]["scale"]))
    # end-of-step scales: the 16-commit window spans two steps, so the spike of step 5 holds the scale down through
    # step 6 and has rolled out by the end of step 7; the one-step collapse at step 9 never owns a whole window (its
    # tensors are cast with the neighbours' scale and land in FP8 subnormals and zeros, which the byte checks cover)
    assert scales[5] < scales[4] / 50 and scales[6] < scales[4] / 50
    assert scales[7] > scales[6] * 10
    assert 0.2 < scales[10] / scales[8] < 5
    st = S.G[0].state()
    assert st["classes"]["X"]["count"] == 96 and st["classes"]["W"]["count"] == 12 and st["e_W"] == 12


def test_config5_direct_placement_against_staged_and_oracle(qe):
    # 48 small linears accumulating into one flat 48 x 2^20 buffer at offsets i * 2^20, 32 microbatches.
    ref = None
    for mode in (qe.EAGER, qe.GRAPH):
        for staged in (False, True):
            S = Stage(qe, "C5", mode, with_oracle=False, staged=staged)
            assert S.offsets == [i << 20 for i in range(48)]
            S.run_step(0)
            g = S.grad.cpu().numpy()
            S.boundary()
            if ref is None:
                ref = g
            else:
                assert np.array_equal(ref.view(np.uint32), g.view(np.uint32)), (mode, staged)
    # oracle: three of the linears, every microbatch, full GEMMs
    S = Stage(qe, "C5", qe.GRAPH)
    sel = (0, 17, 47)
    S.run_step(0, heavy=lambda u, m: u in sel, rows=lambda u: (list(range(0, 512, 37)), list(range(1024))), check_state=True)
    for u in sel:
        S.grads_match(u, list(range(1024)), "C5")
    assert np.array_equal(S.grad.cpu().numpy().view(np.uint32), ref.view(np.uint32))
    S.boundary()


# ------------------------------------------------------------------------------------------ config 3 at its stated size
class _OracleFollower:
    """One sampled linear of config 3 followed by the oracle on a thread of its own (the linears are independent, and
    numpy releases the interpreter lock inside its loops, so several followers run side by side while the GPU goes on).
    The driver puts one item per action of that linear, in order; every item carries what the GPU produced (state after
    the action, and for heavy actions FP8 bytes and output rows), which is compared here."""

    def __init__(self, name, T, K, N, H, P, unit, rows_T, rows_N):
        import queue
        import threading

        self.name, self.rows_T, self.rows_N = name, rows_T, rows_N
        self.O = OracleLinear(T, K, N, H, 0, P, unit=unit)
        self.buf = np.zeros(N * K, np.float32)  # untouched pages stay uncommitted: only sampled rows are written
        self.absp = 0.0
        self.tapes = {}
        self.q = queue.Queue(maxsize=4)
        self.error = None
        self.checked = {"state": 0, "bytes": 0, "gemm_rows": 0, "grad_rows": 0}
        self.t = threading.Thread(target=self._loop, daemon=True)
        self.t.start()

    def put(self, *item):
        self.q.put(item)

    def finish(self):
        self.q.put(None)
        self.t.join()
        if self.error:
            raise AssertionError(f"oracle follower {self.name}: {self.error}")

    def _loop(self):
        import traceback

        while True:
            item = self.q.get()
            if item is None:
                return
            if self.error:
                continue  # keep draining so that the driver never blocks
            try:
                self._do(*item)
            except Exception:  # noqa: BLE001
                self.error = traceback.format_exc()

    def _state(self, g, what):
        assert g["device_status"] == 0 and g["device_token"] == g["token"], what
        assert state_equal_except_Y(g, self.O.state()), what
        self.checked["state"] += 1

    def _do(self, kind, step, m, *a):
        O, what = self.O, (self.name, kind, step, m)
        if kind == "W":
            O.set_weight(a[0])
        elif kind == "F":
            x_bits, tape, g, heavy = a
            self.tapes[m], oy = O.forward(m, O.e_W, x_bits, rows=self.rows_T, light=heavy is None)
            assert tape == (tuple(self.tapes[m].key), tuple(self.tapes[m].ref)), what
            self._state(g, what)
            if heavy is not None:
                slot = O.slots[self.tapes[m].ref.slot]
                assert np.array_equal(heavy["Xq"], slot.Xq), ("Xq",) + what
                assert np.array_equal(heavy["Wq"], O.Wq), ("Wq",) + what
                assert g["slot_sinv_X"][self.tapes[m].ref.slot].view(np.uint32) == np.float32(slot.sinv_X).view(np.uint32)
                assert_gemm_close(heavy["rows"], oy, ("Y",) + what)
                self.checked["bytes"] += 2
                self.checked["gemm_rows"] += len(self.rows_T)
        elif kind == "dI":
            dy_bits, g, heavy = a
            odx = O.backward_dI(self.tapes[m], dy_bits, rows=self.rows_T, light=heavy is None)
            self._state(g, what)
            if heavy is not None:
                slot = O.slots[self.tapes[m].ref.slot]
                assert np.array_equal(heavy["Gq"], slot.Gq), ("Gq",) + what
                assert g["slot_sinv_G"][self.tapes[m].ref.slot].view(np.uint32) == np.float32(slot.sinv_G).view(np.uint32)
                assert_gemm_close(heavy["rows"], odx, ("dX",) + what)
                self.checked["bytes"] += 1
                self.checked["gemm_rows"] += len(self.rows_T)
        elif kind == "dW":
            g, grad_rows = a
            slot = O.slots[self.tapes[m].ref.slot]
            if slot.Xq is not None and slot.Gq is not None:
                if m == 0:
                    self.absp = 0.0
                self.absp = self.absp + dW_abs_products(slot, self.rows_N)
            O.backward_dW(self.tapes.pop(m), self.buf, 0, rows=self.rows_N)
            self._state(g, what)
            if grad_rows is not None:  # every microbatch up to this one was heavy: the slice's rows so far
                want = self.buf.reshape(O.N, O.K)[self.rows_N]
                assert_grad_close(grad_rows, want, ("main_grad",) + what, abs_products=self.absp, rel_tol=1e-5, contraction=O.T)
                self.checked["grad_rows"] += len(self.rows_N)
        elif kind == "boundary":
            O.optimizer_boundary(a[0])
            self._state(a[1], what)


def _one_row_per_tile(n, mul):
    """One row in every 128-row tile (so every 256-row tile pair, every wave and both CTAs of a pair are visited)."""
    return [128 * i + (mul * i + 7) % 128 for i in range(n // 128)]


def test_config3_four_layers_sixteen_microbatches_ten_steps_replayed(qe):
    """Config 3 as stated: Llama-3-8B shapes (T = 4096; qkv 4096->6144, o 4096->4096, gate/up 4096->28672, down
    14336->4096), 4 layers, 16 microbatches in zero-bubble order, every F / dI / dW captured once per slot and replayed
    over static buffers for 10 steps with optimizer boundaries between them (Sec. 4.3-4.4), all weight gradients into
    one 3.49 GB flat buffer at the layers' affine offsets.  Inputs are distinct per (step, layer, linear, microbatch),
    drawn by the device generator from the usual seeds; the sampled linears' tensors are copied back for the oracle.

    Checked: (1) step 0 in eager mode against the replayed step 0, bit for bit, every output of every unit at full
    width; (2) the oracle's state after EVERY action of seven sampled linears (all four shapes, all four layers) --
    over all ten steps for six of them; (3) FP8 bytes and GEMM rows (one row per 128-row tile) on heavy units of every
    shape, including a whole step of the attention output projection of every layer, whose complete gradient slice is
    then compared element by element; first-write and first-accumulate gradient rows of the two wide shapes."""
    name = "C3"
    cfg = inputs.CONFIGS[name]
    T, M, steps, nl = cfg["T"], cfg["M"], cfg["steps"], len(cfg["linears"])
    schedule = sched(M, *cfg["sched"])
    P = peak_live(schedule)
    units = [(l, j, K, N) for l in range(cfg["layers"]) for j, (_, K, N) in enumerate(cfg["linears"])]
    offs, per_layer = inputs.grad_offsets(cfg["linears"])
    offsets = [l * per_layer + offs[j] for l, j, _, _ in units]
    assert per_layer == 218103808 and offsets[4:8] == [218103808 + o for o in (0, 25165824, 41943040, 159383552)]
    n = len(units)

    def make(mode):
        ctx = qe.Context(mode)
        W = [inputs.weights(name, l, j, N, K, device=DEV) for l, j, K, N in units]
        G = [qe.Layer(ctx, T, K, N, cfg["H"], cfg["margin"], P, W[u], unit=u) for u, (l, j, K, N) in enumerate(units)]
        grad = torch.full((per_layer * cfg["layers"],), 3.0, device=DEV)  # stale contents: microbatch 0 must overwrite
        return ctx, W, G, grad

    # ---- (1a) step 0, eager: keep every output on the device
    ctx, W, G, grad = make(qe.EAGER)
    eager = {}
    tapes = {}
    for a, m in schedule:
        for u in (range(n) if a == "F" else range(n - 1, -1, -1)):
            l, j, K, N = units[u]
            if a == "F":
                y = torch.empty((T, N), dtype=torch.bfloat16, device=DEV)
                tapes[(u, m)] = G[u].forward(m, 0, inputs.activations(name, 0, l, j, m, T, K, device=DEV), y)
                eager[(u, m, "Y")] = y
            elif a == "dI":
                dx = torch.empty((T, K), dtype=torch.bfloat16, device=DEV)
                G[u].backward_dI(tapes[(u, m)], inputs.upstream_grads(name, 0, l, j, m, T, N, device=DEV), dx)
                eager[(u, m, "dX")] = dx
            else:
                G[u].backward_dW(tapes[(u, m)], grad, offsets[u])
    torch.cuda.synchronize()
    for L in G:
        L.optimizer_boundary(M)
    eager_grad, eager_state = grad, [L.state() for L in G]
    del G, ctx
    torch.cuda.empty_cache()

    # ---- the ten replayed steps, with the oracle following the sampled linears
    ctx, W, G, grad = make(qe.GRAPH)
    # static buffers: one set per (linear, slot); a forward takes the set of the slot it is about to occupy
    buf = [[{"x": torch.empty((T, K), dtype=torch.bfloat16, device=DEV), "y": torch.empty((T, N), dtype=torch.bfloat16, device=DEV),
             "dy": torch.empty((T, N), dtype=torch.bfloat16, device=DEV), "dx": torch.empty((T, K), dtype=torch.bfloat16, device=DEV)}
            for _ in range(P)] for _, _, K, N in units]
    rows_T = _one_row_per_tile(T, 37)
    U = lambda l, j: l * nl + j
    # sampled linear -> (steps followed, heavy (step, mb) units, (step, mb) after whose dW the gradient rows are compared)
    all_mb = lambda st: {(st, m) for m in range(M)}
    plan = {
        U(0, 0): (steps, {(0, 0), (9, 15)}, {(0, 0)}),                      # qkv, layer 0
        U(0, 1): (steps, all_mb(0), {(0, M - 1)}),                          # o, every layer: one whole heavy step each
        U(1, 1): (steps, all_mb(3), {(3, M - 1)}),
        U(2, 1): (steps, all_mb(6), {(6, M - 1)}),
        U(3, 1): (steps, all_mb(9), {(9, M - 1)}),
        U(2, 3): (steps, {(0, 0), (0, 1), (9, 15)}, {(0, 0), (0, 1)}),      # down, layer 2
        U(3, 2): (1, {(0, 0), (0, 1)}, {(0, 0), (0, 1)}),                   # gate/up, layer 3: first step only
    }
    followers = {}
    for u, (nsteps, heavy, gchk) in plan.items():
        l, j, K, N = units[u]
        followers[u] = _OracleFollower(f"layer {l} {cfg['linears'][j][0]}", T, K, N, cfg["H"], P, u, rows_T, _one_row_per_tile(N, 53))
    bits = lambda t: inputs.bits(t.cpu())
    compared = 0
    for step in range(steps):
        for u, (l, j, K, N) in enumerate(units):
            if step > 0:
                W[u] = inputs.optimizer_perturbation(W[u], name, step, l, j)
                G[u].weight.copy_(W[u])
            if u in plan and step < plan[u][0]:
                followers[u].put("W", step, -1, bits(W[u]))
        tapes = {}
        for a, m in schedule:
            for u in (range(n) if a == "F" else range(n - 1, -1, -1)):
                l, j, K, N = units[u]
                L = G[u]
                f = followers[u] if (u in plan and step < plan[u][0]) else None
                heavy = f is not None and (step, m) in plan[u][1]
                if a == "F":
                    b = buf[u][L.next_slot()]
                    b["x"].copy_(inputs.activations(name, step, l, j, m, T, K, device=DEV))
                    tapes[(u, m)] = t = L.forward(m, step, b["x"], b["y"])
                    assert buf[u][t.ref.slot] is b
                    if step == 0:
                        assert torch.equal(b["y"].view(torch.int16), eager.pop((u, m, "Y")).view(torch.int16)), ("replay != eager: Y", u, m)
                        compared += 1
                    if f:
                        h = {"Xq": L.read_fp8(0, t.ref.slot), "Wq": L.read_fp8(4), "rows": bits(b["y"][rows_T])} if heavy else None
                        f.put("F", step, m, bits(b["x"]), t.astuple(), L.state(), h)
                elif a == "dI":
                    t = tapes[(u, m)]
                    b = buf[u][t.ref.slot]
                    b["dy"].copy_(inputs.upstream_grads(name, step, l, j, m, T, N, device=DEV))
                    L.backward_dI(t, b["dy"], b["dx"])
                    if step == 0:
                        assert torch.equal(b["dx"].view(torch.int16), eager.pop((u, m, "dX")).view(torch.int16)), ("replay != eager: dX", u, m)
                        compared += 1
                    if f:
                        h = {"Gq": L.read_fp8(2, t.ref.slot), "rows": bits(b["dx"][rows_T])} if heavy else None
                        f.put("dI", step, m, bits(b["dy"]), L.state(), h)
                else:
                    L.backward_dW(tapes[(u, m)], grad, offsets[u])
                    if f:
                        g_rows = None
                        if (step, m) in plan[u][2]:
                            g_rows = grad[offsets[u]: offsets[u] + N * K].view(N, K)[f.rows_N].cpu().numpy()
                        f.put("dW", step, m, L.state(), g_rows)
            assert not any(f.error for f in followers.values()), [f.error for f in followers.values() if f.error][0]
        torch.cuda.synchronize()
        for u, L in enumerate(G):
            L.optimizer_boundary(M)
            if u in plan and step < plan[u][0]:
                followers[u].put("boundary", step, -1, M, L.state())
        if step == 0:
            assert compared == 2 * n * M and not eager
            assert torch.equal(grad.view(torch.int32), eager_grad.view(torch.int32)), "replay != eager: main_grad"
            for x, y in zip(eager_state, [L.state() for L in G]):
                assert state_equal({**x, "slots": []}, {**y, "slots": []}) and x["device_token"] == y["device_token"]
            del eager_grad
            torch.cuda.empty_cache()
    for f in followers.values():
        f.finish()
    st = ctx.stats()
    assert st["graphs_built"] == n * (3 * P + 1) and st["eager_launches"] == 0  # G_r = 3 P L (+ one refresh graph per linear)
    assert st["graph_replays"] == steps * n * (3 * M + 1)
    for L in G:
        s_ = L.state()
        assert s_["e_W"] == steps and s_["token"] == steps * 2 * M and s_["device_status"] == 0
    total = {k: sum(f.checked[k] for f in followers.values()) for k in ("state", "bytes", "gemm_rows", "grad_rows")}
    assert total["state"] == sum((3 * M + 1) * plan[u][0] for u in plan)
    assert total["bytes"] >= 3 * (4 * M + 7) and total["grad_rows"] > 0
