#include "psa_internal.h"
namespace psa {
psa_status_t launch_bwd(const psa_plan_t*, const void*, const void*, const void*, const void*, const void*,
                        const float*, void*, void*, void*, void*, int32_t*, void*) {
  return PSA_ERR_UNSUPPORTED;
}
}  // namespace psa
