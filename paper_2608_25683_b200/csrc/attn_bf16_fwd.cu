#include "kernels.h"
namespace psrl {
psrl_status_t fwd_bf16(const AttnArgs&) { return PSRL_ERR_UNSUPPORTED; }
}
