// placeholder until the tcgen05 chain lands
#include "im_internal.h"
#include "mlp.h"
namespace im {
im_status tc_policy_create(im_policy *, const void *const *, const float *const *) { return IM_ERR_UNSUPPORTED; }
void tc_policy_destroy(im_policy *) {}
im_status tc_policy_forward(im_policy *, uint32_t, int32_t, const float *, int32_t, float *, float *, float *) { return IM_ERR_UNSUPPORTED; }
}
