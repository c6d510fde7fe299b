// Tensor-core (tcgen05 / TMEM) Gram-form kernel.  Placeholder until the kernel lands: reports
// that no shape is covered, so every call is served by the direct-difference kernels.
#include "fd_internal.h"

namespace fd {

bool tc_supported(const fd_ctx*, const ApplyArgs&) { return false; }

fd_status apply_tc(fd_ctx* c, const ApplyArgs&) {
    return fail(c, FD_ERR_UNSUPPORTED, "tensor-core path not built");
}

}  // namespace fd
