// mwu_keep_n_of_m: of every four consecutive weights of a row keep the n of largest magnitude
// (Section 4.7: "1x4 blocks with 50 % prune ratio in each block", the pattern sparse tensor cores
// take), and mwu_gemm_dense: the two-operand tensor-core GEMM on a dense bf16 weight matrix, which
// is how the result is multiplied here (the kept / dropped pattern saves storage, not FLOPs: the
// product runs on the dense tensor-core path).
#include "mwu_gemm_dev.cuh"

namespace mwu {
namespace gemm {
EncodeTiledFn get_encode_fn();          // mwu_gemm.cu
cudaError_t launch_dense(const CUtensorMap &tmap_x, const CUtensorMap &tmap_w, const CUtensorMap &tmap_y,
                         const Params &p, int sm_count, cudaStream_t st);
}  // namespace gemm

namespace nm {

// One thread per group of four weights: coalesced 16-byte loads and stores.  Weight l stays when
// fewer than n others of its group come before it in the order (magnitude descending, index
// ascending).  Eight neighbouring threads assemble one word of the keep bitmap.
__global__ void __launch_bounds__(256) keep_n_of_4_kernel(const float *W, const float *U, long long n_groups, int n,
                                                          float *Q, unsigned *keep_bits, unsigned short *Wd,
                                                          long long cols, long long ldw, unsigned *dev_status) {
    const long long n_iter = (n_groups + 7) / 8 * 8;          // whole octets of threads take part in the shuffles
    unsigned bad = 0;
    for (long long g = (long long)blockIdx.x * blockDim.x + threadIdx.x; g < n_iter;
         g += (long long)gridDim.x * blockDim.x) {
        const bool live = g < n_groups;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (live) {
            v = __ldg(reinterpret_cast<const float4 *>(W) + g);
            if (U) {
                const float4 d = __ldg(reinterpret_cast<const float4 *>(U) + g);
                v.x = __fadd_rn(v.x, d.x); v.y = __fadd_rn(v.y, d.y); v.z = __fadd_rn(v.z, d.z); v.w = __fadd_rn(v.w, d.w);
            }
        }
        const float x[4] = {v.x, v.y, v.z, v.w};
        float a[4];
        unsigned keep = 0;
#pragma unroll
        for (int l = 0; l < 4; ++l) {
            a[l] = fabsf(x[l]);
            bad |= (__float_as_uint(a[l]) >= 0x7f800000u) ? 1u : 0u;
        }
#pragma unroll
        for (int l = 0; l < 4; ++l) {
            int before = 0;
#pragma unroll
            for (int o = 0; o < 4; ++o)
                if (o != l) before += (a[o] > a[l] || (a[o] == a[l] && o < l)) ? 1 : 0;
            keep |= (before < n ? 1u : 0u) << l;
        }
        float q[4];
#pragma unroll
        for (int l = 0; l < 4; ++l) q[l] = ((keep >> l) & 1u) ? x[l] : 0.f;
        if (live) {
            if (Q) reinterpret_cast<float4 *>(Q)[g] = make_float4(q[0], q[1], q[2], q[3]);
            if (Wd) {
                const long long f = g * 4, row = f / cols, col = f - row * cols;
                const __nv_bfloat162 h0 = __floats2bfloat162_rn(q[0], q[1]), h1 = __floats2bfloat162_rn(q[2], q[3]);
                *reinterpret_cast<uint2 *>(Wd + row * ldw + col) =
                    make_uint2(*reinterpret_cast<const unsigned *>(&h0), *reinterpret_cast<const unsigned *>(&h1));
            }
        }
        unsigned word = (live ? keep : 0u) << (4 * (threadIdx.x & 7));
        word |= __shfl_xor_sync(0xffffffffu, word, 1);
        word |= __shfl_xor_sync(0xffffffffu, word, 2);
        word |= __shfl_xor_sync(0xffffffffu, word, 4);
        if ((threadIdx.x & 7) == 0 && live) keep_bits[g >> 3] = word;
    }
    if (bad) atomicOr(dev_status, (unsigned)MWU_DEV_NONFINITE);
}

}  // namespace nm
}  // namespace mwu

extern "C" int mwu_keep_n_of_m(int64_t rows, int64_t cols, int32_t n, int32_t m, const float *W,
                               const float *U_dual, float *Q, uint32_t *keep_bits, void *Wd, int64_t ldw,
                               uint32_t *dev_status, void *cuda_stream) {
    using namespace mwu;
    if (!W || !keep_bits || !dev_status) return MWU_ERR_INVALID_ARG;
    if (rows <= 0 || cols <= 0 || m != 4 || n < 0 || n > 4 || cols % 4 != 0) return MWU_ERR_SHAPE;
    if (rows * cols >= (int64_t(1) << 40)) return MWU_ERR_SHAPE;
    if (Wd && ldw < cols) return MWU_ERR_SHAPE;
    if (!aligned_to(W, 16) || !aligned_to(U_dual, 16) || !aligned_to(Q, 16) || !aligned_to(keep_bits, 4) ||
        !aligned_to(Wd, 16) || (Wd && ldw % 8 != 0) || !aligned_to(dev_status, 4))
        return MWU_ERR_ALIGNMENT;
    int sm_count = 0;
    const int rc = check_device(&sm_count);
    if (rc != MWU_OK) return rc;
    const long long n_groups = rows * cols / 4;
    const long long want = (n_groups + 255) / 256;
    const long long cap = (long long)sm_count * 16;
    const int grid = (int)(want < cap ? want : cap);
    nm::keep_n_of_4_kernel<<<grid, 256, 0, (cudaStream_t)cuda_stream>>>(W, U_dual, n_groups, n, Q, keep_bits,
                                                                       (unsigned short *)Wd, cols, ldw, dev_status);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? MWU_OK : MWU_ERR_CUDA;
}

extern "C" int mwu_gemm_dense(int64_t rows, int64_t cols, const void *Wd, int64_t ldw, const void *X, int64_t M,
                              int64_t ldx, void *Y, int64_t ldy, int32_t y_dtype, uint32_t *dev_status,
                              void *cuda_stream) {
    using namespace mwu;
    using namespace mwu::gemm;
    if (!Wd || !X || !Y || !dev_status || M < 0) return MWU_ERR_INVALID_ARG;
    if (y_dtype != 0 && y_dtype != 1) return MWU_ERR_INVALID_ARG;
    if (rows <= 0 || cols <= 0 || ldw < cols || ldx < cols || ldy < rows) return MWU_ERR_SHAPE;
    if (M >= (int64_t(1) << 31) || ldx >= (int64_t(1) << 31) || rows >= (int64_t(1) << 31)) return MWU_ERR_SHAPE;
    if (!aligned_to(Wd, 16) || !aligned_to(X, 16) || !aligned_to(Y, 16) || ldw % 8 != 0 || ldx % 8 != 0 ||
        ldy % (y_dtype ? 4 : 8) != 0 || !aligned_to(dev_status, 4))
        return MWU_ERR_ALIGNMENT;
    if (M == 0) return MWU_OK;
    int sm_count = 0;
    const int rc = check_device(&sm_count);
    if (rc != MWU_OK) return rc;
    EncodeTiledFn encode = get_encode_fn();
    if (!encode) return MWU_ERR_CUDA;
    Params p = {};
    p.all_live = 1;                                     // no packed record table: every k stage is multiplied
    p.n_rec_tiles = (rows + kTileRows - 1) / kTileRows;
    p.n_stages = (cols + BK - 1) / BK;
    if (p.n_stages > MAX_STAGES_K) return MWU_ERR_SHAPE;
    p.M = M; p.N = rows; p.K = cols;
    p.Y = Y; p.ldy = ldy; p.y_fp32 = y_dtype;
    p.dev_status = dev_status;
    auto enc2d = [&](CUtensorMap *tm, const void *ptr, int64_t inner, int64_t outer, int64_t ld, int box_rows) {
        const cuuint64_t gdim[2] = {(cuuint64_t)inner, (cuuint64_t)outer};
        const cuuint64_t gstride[1] = {(cuuint64_t)ld * 2};
        const cuuint32_t box[2] = {(cuuint32_t)BK, (cuuint32_t)box_rows};
        const cuuint32_t estr[2] = {1, 1};
        return encode(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(ptr), gdim, gstride, box, estr,
                      CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
    };
    CUtensorMap tmap_x, tmap_w;
    if (!enc2d(&tmap_x, X, cols, M, ldx, BMH) || !enc2d(&tmap_w, Wd, cols, rows, ldw, kTileRows)) return MWU_ERR_CUDA;
    CUtensorMap tmap_y = tmap_x;
    if (y_dtype == 0) {
        if (!enc2d(&tmap_y, Y, rows, M, ldy, 32)) return MWU_ERR_CUDA;
        p.y_tma = 1;
    }
    return launch_dense(tmap_x, tmap_w, tmap_y, p, sm_count, (cudaStream_t)cuda_stream) == cudaSuccess ? MWU_OK
                                                                                                       : MWU_ERR_CUDA;
}
