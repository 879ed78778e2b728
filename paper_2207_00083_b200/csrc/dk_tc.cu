// Tensor-core path (tcgen05 / TMEM / TMA).
#include "dk_internal.h"

namespace dk {

dk_status tc_init(dk_ctx* ctx) { ctx->tc_state = nullptr; return DK_OK; }
void tc_destroy(dk_ctx*) {}

}  // namespace dk
