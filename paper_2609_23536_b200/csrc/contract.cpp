// Contract core.  Every rule cites the part of the paper it enforces; a failed check changes nothing
// (Algorithm 1: a check precedes its action, the transition commits only after the action succeeded).
#include "contract.h"

#include <cstring>
#include <new>
#include <vector>

#include "error.h"

using qe::fail;

static bool key_eq(const qe_tape_key& a, const qe_tape_key& b) {
  return a.epoch == b.epoch && a.stage == b.stage && a.mb == b.mb && a.unit == b.unit && a.inv == b.inv;
}

uint32_t qe_contract::live_tapes() const {
  uint32_t n = 0;
  for (uint32_t p = 0; p < P; ++p) n += slot[p].live ? 1u : 0u;
  return n;
}

int qe_contract::lowest_free() const {
  for (uint32_t p = 0; p < P; ++p)
    if (!slot[p].live) return (int)p;
  return -1;
}

// Invariant 2: dereferencing verifies generation equality (no stale read, no ABA across slot reuse).
int32_t qe_contract::resolve(const qe_tape* t, uint32_t* p_out) const {
  if (!t) return fail(QE_ERR_BAD_ARG, "tape is null");
  const uint32_t p = t->ref.slot;
  if (p >= P) return fail(QE_ERR_STALE_REF, "slot %u out of range", p);
  const Slot& s = slot[p];
  if (!s.live || s.gen != t->ref.gen)
    return fail(QE_ERR_STALE_REF, "slot %u: reference generation %llu, slot generation %llu, live %d", p,
                (unsigned long long)t->ref.gen, (unsigned long long)s.gen, (int)s.live);
  if (!key_eq(s.key, t->key)) return fail(QE_ERR_KEY_MISMATCH, "slot %u holds a different key", p);
  if ((uint64_t)t->key.epoch != (e_W & 0xffffffffull)) return fail(QE_ERR_EPOCH, "tape epoch %u, e_W %llu", t->key.epoch, (unsigned long long)e_W);
  *p_out = p;
  return QE_OK;
}

extern "C" {

int32_t qe_registry_create(qe_registry** out) {
  if (!out) return fail(QE_ERR_BAD_ARG, "out is null");
  *out = new (std::nothrow) qe_registry();
  if (!*out) return fail(QE_ERR_BAD_ARG, "out of host memory");
  (*out)->state = std::make_shared<qe::RegistryState>();
  return QE_OK;
}
int32_t qe_registry_destroy(qe_registry* r) {
  delete r;
  return QE_OK;
}

int32_t qe_contract_create(uint32_t slots, uint32_t stage, uint32_t unit, uint32_t inv, qe_registry* registry,
                           qe_contract** out) {
  if (!out) return fail(QE_ERR_BAD_ARG, "out is null");
  if (slots < 1 || slots > QE_MAX_SLOTS) return fail(QE_ERR_BAD_ARG, "slots %u not in [1, %u]", slots, QE_MAX_SLOTS);
  qe_contract* c = new (std::nothrow) qe_contract();
  if (!c) return fail(QE_ERR_BAD_ARG, "out of host memory");
  c->P = slots;
  c->stage = stage;
  c->unit = unit;
  c->inv = inv;
  if (registry) c->registry = registry->state;
  *out = c;
  return QE_OK;
}

int32_t qe_contract_destroy(qe_contract* c) {
  if (c && c->registry) {
    std::lock_guard<std::mutex> g(c->registry->mu);
    c->registry->bound.erase(c);
  }
  delete c;
  return QE_OK;
}

// Sec. 3.3 / Invariant 3: every forward requires parameter-epoch consistency; the first forward of an epoch
// refreshes the cache, later ones verify it.  Eq. 1-2: one live tape per key, lowest free slot, no pre-emption.
int32_t qe_contract_forward_check(const qe_contract* c, uint32_t mb, uint64_t gen, int32_t* refresh_out,
                                  uint32_t* slot_out) {
  if (!c) return fail(QE_ERR_BAD_ARG, "contract is null");
  if (c->aborted) return fail(QE_ERR_ABORTED, "step aborted; rebuild the arena first");
  if (mb >= QE_MAX_MICROBATCHES) return fail(QE_ERR_BAD_ARG, "microbatch %u >= %u", mb, QE_MAX_MICROBATCHES);
  if (gen != c->e_W) return fail(QE_ERR_EPOCH, "caller weight version %llu, e_W %llu", (unsigned long long)gen, (unsigned long long)c->e_W);
  const bool refresh = c->fwd_in_epoch == 0;
  if (!refresh && c->e_C != c->e_W) return fail(QE_ERR_STALE_CACHE, "cache refresh required (e_C != e_W)");
  qe_tape_key key{(uint32_t)c->e_W, c->stage, mb, c->unit, c->inv};
  for (uint32_t p = 0; p < c->P; ++p)
    if (c->slot[p].live && key_eq(c->slot[p].key, key)) return fail(QE_ERR_KEY_LIVE, "key already live in slot %u", p);
  const int p = c->lowest_free();
  if (p < 0) return fail(QE_ERR_POOL_FULL, "all %u slots occupied", c->P);
  if (refresh_out) *refresh_out = refresh ? 1 : 0;
  if (slot_out) *slot_out = (uint32_t)p;
  return QE_OK;
}

int32_t qe_contract_forward_commit(qe_contract* c, uint32_t mb, qe_tape* tape_out) {
  int32_t refresh = 0;
  uint32_t p = 0;
  int32_t st = qe_contract_forward_check(c, mb, c ? c->e_W : 0, &refresh, &p);
  if (st != QE_OK) return st;
  qe_contract::Slot& s = c->slot[p];
  s.gen += 1;  // monotone across reuse
  s.live = true;
  s.bits = 0;
  s.key = qe_tape_key{(uint32_t)c->e_W, c->stage, mb, c->unit, c->inv};
  if (refresh) c->e_C = c->e_W;
  c->token += 1;  // Invariant 1: F advances the effect token
  c->fwd_in_epoch += 1;
  if (tape_out) {
    std::memset(tape_out, 0, sizeof(*tape_out));
    tape_out->key = s.key;
    tape_out->ref.slot = p;
    tape_out->ref.gen = s.gen;
  }
  return QE_OK;
}

int32_t qe_contract_dI_check(const qe_contract* c, const qe_tape* t) {
  if (!c) return fail(QE_ERR_BAD_ARG, "contract is null");
  if (c->aborted) return fail(QE_ERR_ABORTED, "step aborted");
  uint32_t p;
  int32_t st = c->resolve(t, &p);
  if (st != QE_OK) return st;
  if (c->slot[p].bits & qe::kDIBit) return fail(QE_ERR_DUP_CONSUME, "dI already consumed slot %u", p);
  return QE_OK;
}

int32_t qe_contract_dI_commit(qe_contract* c, const qe_tape* t) {
  int32_t st = qe_contract_dI_check(c, t);
  if (st != QE_OK) return st;
  c->slot[t->ref.slot].bits |= qe::kDIBit;
  c->token += 1;  // Invariant 1: dI advances the effect token; dW never does
  return QE_OK;
}

// Sec. 3.4: destination validated; microbatch 0 initialises; duplicate / aliased writes fail.
int32_t qe_contract_dW_check(const qe_contract* c, const qe_tape* t, uint64_t dest_addr, uint64_t dest_elems,
                             uint64_t offset, uint64_t slice_elems, int32_t* accumulate_out) {
  if (!c) return fail(QE_ERR_BAD_ARG, "contract is null");
  if (c->aborted) return fail(QE_ERR_ABORTED, "step aborted; arena unusable for this epoch");
  uint32_t p;
  int32_t st = c->resolve(t, &p);
  if (st != QE_OK) return st;
  const qe_contract::Slot& s = c->slot[p];
  if (s.bits & qe::kDWBit) return fail(QE_ERR_DUP_CONSUME, "dW already consumed slot %u", p);
  if (!(s.bits & qe::kDIBit)) return fail(QE_ERR_ORDER, "dW before dI on slot %u", p);
  if (dest_addr == 0) return fail(QE_ERR_DEST, "destination is null");
  if (offset > dest_elems || slice_elems > dest_elems - offset)
    return fail(QE_ERR_DEST, "slice [%llu, +%llu) exceeds buffer of %llu elements", (unsigned long long)offset,
                (unsigned long long)slice_elems, (unsigned long long)dest_elems);
  const uint64_t lo = dest_addr + 4ull * offset, hi = lo + 4ull * slice_elems;
  if (lo % 16 != 0) return fail(QE_ERR_DEST, "destination slice not 16-byte aligned");
  if (c->has_dest && (c->dest_addr != dest_addr || c->dest_off != offset))
    return fail(QE_ERR_DEST, "differs from the destination bound for this epoch");
  if (c->registry) {
    std::lock_guard<std::mutex> g(c->registry->mu);
    for (const auto& kv : c->registry->bound)
      if (kv.first != c && kv.second.lo < hi && lo < kv.second.hi)
        return fail(QE_ERR_DEST, "destination aliases another layer's slice");
  }
  const uint32_t mb = t->key.mb;
  if ((c->write_mask >> mb) & 1ull) return fail(QE_ERR_DUP_WRITE, "microbatch %u already wrote this epoch", mb);
  if (c->write_mask == 0 && mb != 0) return fail(QE_ERR_ORDER, "first write of the epoch must be microbatch 0, got %u", mb);
  if (accumulate_out) *accumulate_out = c->write_mask == 0 ? 0 : 1;
  return QE_OK;
}

int32_t qe_contract_dW_commit(qe_contract* c, const qe_tape* t, uint64_t dest_addr, uint64_t offset,
                              uint64_t slice_elems) {
  // re-validate everything that does not depend on the buffer length (already checked before the action)
  int32_t st = qe_contract_dW_check(c, t, dest_addr, UINT64_MAX, offset, slice_elems, nullptr);
  if (st != QE_OK) return st;
  c->has_dest = true;
  c->dest_addr = dest_addr;
  c->dest_off = offset;
  if (c->registry) {
    std::lock_guard<std::mutex> g(c->registry->mu);
    const uint64_t lo = dest_addr + 4ull * offset;
    c->registry->bound[c] = qe::RegistryState::Range{lo, lo + 4ull * slice_elems};
  }
  qe_contract::Slot& s = c->slot[t->ref.slot];
  c->write_mask |= 1ull << t->key.mb;
  s.bits |= qe::kDWBit;
  s.live = false;  // both consumers done: release; the generation stays (Eq. 2)
  return QE_OK;
}

// Algorithm 1, after the action loop.
int32_t qe_contract_boundary_check(const qe_contract* c, uint32_t expected) {
  if (!c) return fail(QE_ERR_BAD_ARG, "contract is null");
  if (c->aborted) return fail(QE_ERR_ABORTED, "step aborted");
  if (expected < 1 || expected > QE_MAX_MICROBATCHES) return fail(QE_ERR_BAD_ARG, "microbatches_expected %u", expected);
  if (c->live_tapes()) return fail(QE_ERR_PENDING, "%u live tape(s) at the optimizer boundary", c->live_tapes());
  const uint64_t want = expected == 64 ? ~0ull : ((1ull << expected) - 1);
  if (c->write_mask != want)
    return fail(QE_ERR_INCOMPLETE, "gradient write mask %#llx, expected %#llx", (unsigned long long)c->write_mask, (unsigned long long)want);
  return QE_OK;
}

int32_t qe_contract_boundary(qe_contract* c, uint32_t expected) {
  const int32_t st = qe_contract_boundary_check(c, expected);
  if (st != QE_OK) return st;
  c->e_W += 1;
  c->write_mask = 0;
  c->fwd_in_epoch = 0;
  c->has_dest = false;
  if (c->registry) {
    std::lock_guard<std::mutex> g(c->registry->mu);
    c->registry->bound.erase(c);
  }
  return QE_OK;
}

// Sec. 3.1 / 4.5: an aborted step purges outstanding tapes of epoch e; the arena is flagged unusable.
int32_t qe_contract_abort(qe_contract* c) {
  if (!c) return fail(QE_ERR_BAD_ARG, "contract is null");
  for (uint32_t p = 0; p < c->P; ++p)
    if (c->slot[p].live && c->slot[p].key.epoch == (uint32_t)c->e_W) c->slot[p].live = false;
  c->aborted = true;
  return QE_OK;
}

int32_t qe_contract_rebuild(qe_contract* c) {
  if (!c) return fail(QE_ERR_BAD_ARG, "contract is null");
  if (c->live_tapes()) return fail(QE_ERR_PENDING, "live tape during rebuild");
  c->aborted = false;
  c->write_mask = 0;
  c->fwd_in_epoch = 0;
  c->has_dest = false;
  if (c->registry) {
    std::lock_guard<std::mutex> g(c->registry->mu);
    c->registry->bound.erase(c);
  }
  return QE_OK;
}

int32_t qe_contract_invalidate_cache(qe_contract* c) {
  if (!c) return fail(QE_ERR_BAD_ARG, "contract is null");
  c->e_C = QE_INVALID_EPOCH;
  return QE_OK;
}

int32_t qe_contract_checkpoint_check(const qe_contract* c) {
  if (!c) return fail(QE_ERR_BAD_ARG, "contract is null");
  if (c->live_tapes()) return fail(QE_ERR_PENDING, "checkpoint withheld: %u live tape(s)", c->live_tapes());
  return QE_OK;
}

int32_t qe_contract_restore(qe_contract* c, uint64_t e_W) {
  if (!c) return fail(QE_ERR_BAD_ARG, "contract is null");
  if (c->live_tapes()) return fail(QE_ERR_PENDING, "restore with %u live tape(s)", c->live_tapes());
  c->e_W = e_W;
  c->e_C = QE_INVALID_EPOCH;  // cache contents are process-local: refresh on the first forward
  c->fwd_in_epoch = 0;
  c->write_mask = 0;
  c->aborted = false;
  c->has_dest = false;
  if (c->registry) {
    std::lock_guard<std::mutex> g(c->registry->mu);
    c->registry->bound.erase(c);
  }
  return QE_OK;
}

int32_t qe_contract_get(const qe_contract* c, qe_contract_view* v) {
  if (!c || !v) return fail(QE_ERR_BAD_ARG, "null argument");
  std::memset(v, 0, sizeof(*v));
  v->e_W = c->e_W;
  v->e_C = c->e_C;
  v->token = c->token;
  v->write_mask = c->write_mask;
  v->fwd_in_epoch = c->fwd_in_epoch;
  v->aborted = c->aborted ? 1u : 0u;
  v->slots = c->P;
  v->live_tapes = c->live_tapes();
  for (uint32_t p = 0; p < c->P; ++p) {
    v->slot[p].gen = c->slot[p].gen;
    v->slot[p].live = c->slot[p].live ? 1u : 0u;
    v->slot[p].bits = c->slot[p].bits;
    v->slot[p].key = c->slot[p].key;
  }
  return QE_OK;
}

// ---- issue plan of a whole-step action list (host logic only; used by qe_step_run)
int32_t qe_plan_rounds(const qe_step_action* actions, uint32_t n_actions, uint32_t n_layers, uint32_t microbatches,
                       const uint32_t* slots, const uint32_t* live_now, uint32_t window, uint32_t max_group,
                       uint32_t* round_of_action, uint32_t* n_rounds_out) {
  if (!actions || !slots || !round_of_action || !n_rounds_out) return fail(QE_ERR_BAD_ARG, "null argument");
  if (n_actions == 0 || n_layers == 0 || microbatches == 0 || window == 0 || max_group == 0) return fail(QE_ERR_BAD_ARG, "empty list or zero limit");
  const uint32_t M = microbatches;
  struct Unit { uint32_t kind, mb, begin, end; int prev; };
  std::vector<Unit> units;
  std::vector<uint8_t> taken(n_actions, 0);
  int last_of_kind[3] = {-1, -1, -1};
  for (uint32_t i = 0; i < n_actions; ++i) {
    const qe_step_action& a = actions[i];
    if (a.kind > QE_ACT_DW || a.layer >= n_layers || a.mb >= M) return fail(QE_ERR_BAD_ARG, "action %u: kind %u layer %u mb %u", i, a.kind, a.layer, a.mb);
    // a unit: a run of actions of one kind and microbatch over distinct layers
    bool fresh = units.empty() || units.back().kind != a.kind || units.back().mb != a.mb;
    for (uint32_t j = fresh ? i : units.back().begin; !fresh && j < i; ++j) fresh = actions[j].layer == a.layer;
    if (fresh) {
      units.push_back(Unit{a.kind, a.mb, i, i, last_of_kind[a.kind]});
      last_of_kind[a.kind] = (int)units.size() - 1;
    }
    units.back().end = i + 1;
  }
  std::vector<uint8_t> issued((size_t)3 * n_layers * M, 0);  // [kind][layer][mb]
  auto was = [&](uint32_t kind, uint32_t layer, uint32_t mb) -> uint8_t& { return issued[((size_t)kind * n_layers + layer) * M + mb]; };
  std::vector<uint32_t> live(n_layers, 0);
  for (uint32_t l = 0; live_now && l < n_layers; ++l) live[l] = live_now[l];
  size_t first = 0;
  uint32_t round = 0;
  std::vector<uint32_t> group;
  while (first < units.size()) {
    group.clear();
    for (size_t ui = first; ui < units.size() && ui < first + window && group.size() < max_group; ++ui) {
      const Unit& u = units[ui];
      for (uint32_t i = u.begin; i < u.end && group.size() < max_group; ++i) {
        if (taken[i]) continue;
        const qe_step_action& a = actions[i];
        bool ready = true;
        for (uint32_t gi : group)  // one action of a kind per layer, never two of one (layer, microbatch)
          ready = ready && !((actions[gi].kind == a.kind && actions[gi].layer == a.layer) || (actions[gi].layer == a.layer && actions[gi].mb == a.mb));
        if (u.prev >= 0) {  // each layer sees the units of a kind in list order
          const Unit& p = units[u.prev];
          for (uint32_t j = p.begin; j < p.end; ++j)
            if (actions[j].layer == a.layer) ready = ready && taken[j] == 2;
        }
        if (a.kind == QE_ACT_F) ready = ready && live[a.layer] < slots[a.layer];
        if (a.kind == QE_ACT_DI) ready = ready && was(QE_ACT_F, a.layer, a.mb) == 2;
        if (a.kind == QE_ACT_DW) ready = ready && was(QE_ACT_DI, a.layer, a.mb) == 2;
        if (ready) {
          group.push_back(i);
          taken[i] = 1;
        }
        if (a.kind != QE_ACT_DW) break;  // F and dI walk their layers in list order: only the next one can be ready
      }
    }
    if (group.empty()) return fail(QE_ERR_ORDER, "no action of units %zu.. is ready: the list is not a legal schedule for these pools", first);
    for (uint32_t gi : group) {  // visible to later rounds only
      const qe_step_action& a = actions[gi];
      taken[gi] = 2;
      was(a.kind, a.layer, a.mb) = 2;
      if (a.kind == QE_ACT_F) live[a.layer] += 1;
      if (a.kind == QE_ACT_DW && live[a.layer]) live[a.layer] -= 1;
      round_of_action[gi] = round;
    }
    ++round;
    while (first < units.size()) {
      bool all = true;
      for (uint32_t i = units[first].begin; i < units[first].end; ++i) all = all && taken[i] == 2;
      if (!all) break;
      ++first;
    }
  }
  *n_rounds_out = round;
  return QE_OK;
}

}  // extern "C"
