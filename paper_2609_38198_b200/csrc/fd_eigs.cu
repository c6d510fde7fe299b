// Eigensolver, bandwidth flow and out-of-sample extension: placeholders.
#include "fd_internal.h"

extern "C" {

fd_status fd_eigs(fd_ctx* c, int32_t, int32_t, double, int32_t, const float*, int64_t, int32_t, double*, float*, int64_t,
                  fd_eigs_info*) {
    return fd::fail(c, FD_ERR_UNSUPPORTED, "fd_eigs not built");
}

fd_status fd_beta_flow(fd_ctx* c, const fd_flow_opts*, const float*, int64_t, int32_t, fd_probe*, int32_t*, int32_t*,
                       double*, double*, float*, int64_t) {
    return fd::fail(c, FD_ERR_UNSUPPORTED, "fd_beta_flow not built");
}

fd_status fd_nystrom(fd_ctx* c, const float*, int64_t, int64_t, const float*, int64_t, int32_t, const double*, float*,
                     int64_t) {
    return fd::fail(c, FD_ERR_UNSUPPORTED, "fd_nystrom not built");
}

}
