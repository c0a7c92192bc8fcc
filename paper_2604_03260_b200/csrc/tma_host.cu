#include "tma_host.cuh"

#include <cudaTypedefs.h>

namespace focus {

static PFN_cuTensorMapEncodeTiled_v12000 get_encoder() {
    static PFN_cuTensorMapEncodeTiled_v12000 fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(p);
    }
    return fn;
}

int make_tmap_bf16_4d(CUtensorMap* out, const void* base, uint64_t d0, uint64_t d1, uint64_t d2, uint64_t d3,
                      uint64_t s1_bytes, uint64_t s2_bytes, uint64_t s3_bytes, uint32_t box0, uint32_t box1) {
    auto enc = get_encoder();
    if (!enc) return fail(FOCUS_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
    cuuint64_t dims[4] = {d0, d1, d2, d3};
    cuuint64_t strides[3] = {s1_bytes, s2_bytes, s3_bytes};
    cuuint32_t box[4] = {box0, box1, 1, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = enc(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS)
        return fail(FOCUS_ERR_CUDA, "cuTensorMapEncodeTiled failed with CUresult %d (dims %llu %llu %llu %llu)", (int)r,
                    (unsigned long long)d0, (unsigned long long)d1, (unsigned long long)d2, (unsigned long long)d3);
    return FOCUS_OK;
}

int make_tmap_qkv(CUtensorMap* out, const focus_tensor& t, int batch, int H, int n, int D, int rows) {
    // a dimension of extent 1 still needs a legal (multiple of 16 bytes, non-zero) stride
    uint64_t sb = (uint64_t)t.stride_b * 2;
    if (batch == 1) sb = (uint64_t)t.stride_h * 2 * (uint64_t)H;
    return make_tmap_bf16_4d(out, t.ptr, (uint64_t)D, (uint64_t)n, (uint64_t)H, (uint64_t)batch,
                             (uint64_t)t.stride_n * 2, (uint64_t)t.stride_h * 2, sb, 64, (uint32_t)rows);
}

}  // namespace focus
