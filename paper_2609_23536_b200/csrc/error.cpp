#include "error.h"

#include <cstdio>

#include "qe.h"

namespace qe {
static thread_local char g_msg[512] = "";

int32_t fail(int32_t status, const char* fmt, ...) {
  int n = std::snprintf(g_msg, sizeof(g_msg), "%s: ", qe_status_name(status));
  if (n < 0) n = 0;
  va_list ap;
  va_start(ap, fmt);
  std::vsnprintf(g_msg + n, sizeof(g_msg) - n, fmt, ap);
  va_end(ap);
  return status;
}
void clear_error() { g_msg[0] = 0; }
}  // namespace qe

extern "C" const char* qe_last_error(void) { return qe::g_msg; }

extern "C" const char* qe_status_name(int32_t s) {
  switch (s) {
    case QE_OK: return "QE_OK";
    case QE_ERR_BAD_ARG: return "QE_ERR_BAD_ARG";
    case QE_ERR_SHAPE: return "QE_ERR_SHAPE";
    case QE_ERR_KEY_LIVE: return "QE_ERR_KEY_LIVE";
    case QE_ERR_POOL_FULL: return "QE_ERR_POOL_FULL";
    case QE_ERR_STALE_CACHE: return "QE_ERR_STALE_CACHE";
    case QE_ERR_ABORTED: return "QE_ERR_ABORTED";
    case QE_ERR_STALE_REF: return "QE_ERR_STALE_REF";
    case QE_ERR_KEY_MISMATCH: return "QE_ERR_KEY_MISMATCH";
    case QE_ERR_EPOCH: return "QE_ERR_EPOCH";
    case QE_ERR_DUP_CONSUME: return "QE_ERR_DUP_CONSUME";
    case QE_ERR_ORDER: return "QE_ERR_ORDER";
    case QE_ERR_DEST: return "QE_ERR_DEST";
    case QE_ERR_DUP_WRITE: return "QE_ERR_DUP_WRITE";
    case QE_ERR_PENDING: return "QE_ERR_PENDING";
    case QE_ERR_INCOMPLETE: return "QE_ERR_INCOMPLETE";
    case QE_ERR_CUDA: return "QE_ERR_CUDA";
    case QE_ERR_TIMEOUT: return "QE_ERR_TIMEOUT";
    case QE_ERR_WORKSPACE: return "QE_ERR_WORKSPACE";
    case QE_ERR_UNSUPPORTED: return "QE_ERR_UNSUPPORTED";
    default: return "QE_ERR_UNKNOWN";
  }
}

extern "C" uint32_t qe_abi_version(void) { return 1; }
