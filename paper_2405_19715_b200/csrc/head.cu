// Acceptance-prediction head (Eq. 3 / Section 5.1 of arXiv 2405.19715).
#include <cstdio>

#include "specdec_internal.h"

extern "C" int specdec_accept_head(specdec_ctx* ctx, const void*, const specdec_head*, int, int, float*, void*) {
    if (!ctx) return SPECDEC_EINVAL;
    snprintf(ctx->err, sizeof(ctx->err), "accept_head: not built yet");
    return SPECDEC_EUNSUPPORTED;
}
