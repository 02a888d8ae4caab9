// gsd_verify_attn, tcgen05 back end (placeholder until the TMEM kernel lands).
#include "gsd_internal.cuh"
namespace gsd {
int launch_attn_tcgen05(const AttnArgs&) {
    set_error_text("tcgen05 back end not built");
    return GSD_ERR_UNSUPPORTED;
}
}  // namespace gsd
