// Host-only contract core: tape slot pool (TapeKey -> TapeRef with generations), consumer bitmask,
// weight/cache versions, effect-token mirror and gradient-arena write accounting.  No CUDA dependency.
#pragma once
#include <cstdint>
#include <memory>
#include <mutex>
#include <unordered_map>

#include "qe.h"

namespace qe {
struct RegistryState {
  struct Range { uint64_t lo, hi; };  // byte addresses [lo, hi)
  std::mutex mu;
  std::unordered_map<const qe_contract*, Range> bound;
};
}  // namespace qe

// The handle and every contract created with it share ownership of the state, so destroying the handle
// before (or after) the contracts is safe.
struct qe_registry {
  std::shared_ptr<qe::RegistryState> state;
};

struct qe_contract {
  struct Slot {
    uint64_t gen = 0;
    bool live = false;
    uint32_t bits = 0;
    qe_tape_key key{};
  };
  uint32_t P = 0, stage = 0, unit = 0, inv = 0;
  Slot slot[QE_MAX_SLOTS];
  uint64_t e_W = 0, e_C = QE_INVALID_EPOCH, token = 0, write_mask = 0;
  uint32_t fwd_in_epoch = 0;
  bool aborted = false;
  bool has_dest = false;
  uint64_t dest_addr = 0, dest_off = 0;
  std::shared_ptr<qe::RegistryState> registry;

  uint32_t live_tapes() const;
  int lowest_free() const;
  // Retained-work lookup: generation first, then key, then epoch.  Returns QE_OK and the slot index.
  int32_t resolve(const qe_tape* t, uint32_t* p_out) const;
};

namespace qe {
constexpr uint32_t kDIBit = 1u, kDWBit = 2u;
}
