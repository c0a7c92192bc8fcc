// Class-sorted layout of focus_build_tiles (stable sort of tokens by membership-mask value).
#include "common.cuh"

namespace focus {

int launch_build_tiles_sorted(const focus_shape* s, const uint32_t* mq, const uint32_t* mk,
                              const focus_tiles_layout& L, char* ws, cudaStream_t st) {
    (void)s; (void)mq; (void)mk; (void)L; (void)ws; (void)st;
    return fail(FOCUS_ERR_UNSUPPORTED, "class-sorted layout is not built yet");
}

}  // namespace focus
