// Projection for 2- and 3-dim block shapes (Section 3.1; Table 1: [2,2], [2,2,2]).
//
// A block spans dk input channels x dr rows x dt kernel taps of W[rows][cin * taps]; its weights are
// not contiguous in memory, so this path works block by block instead of streaming 64-byte units:
//   shape_stats_kernel     one thread per block gathers its weights and evaluates the fp64 keys of
//                          Section 3.1 (same pairwise tree as the 1-dim kernels, members in
//                          (row, channel, tap) order) into two key arrays.
//   sign_plane_kernel      one bit per weight, v < 0.
//   select_smallest_kernel exact selection of the k smallest (key, index) among the eligible
//                          entries of a key array, as a bitmap: radix selection on the keys' bit
//                          patterns, then the entries holding exactly the threshold key in index order.
//                          Run twice: prune keys of all blocks, then L_u of the blocks not pruned.
//   shape_emit_kernel      one thread per block writes Q, u and, for mwu_admm_step, the dual update
//                          and the residual.
// lower_kernel turns the result of a shape whose blocks are runs of dk entries in each of their rows
// (dt = 1, taps = 1) into the per-row 1-dim arrays mwu_pack reads.
#include "mwu_common.cuh"

namespace mwu {
namespace shapes {

typedef unsigned long long u64;
constexpr int SEL_THREADS = 1024;

struct SParams {
    const float *W;
    const float *U;
    long long rows, cols;
    int dk, dr, dt, taps;
    long long cin_groups, ntg, mb;
    int use_l1;
};

// flat indices of block j's weights in (row, channel, tap) order; returns their number
__device__ __forceinline__ int block_members(const SParams &p, long long j, long long (&idx)[16]) {
    const long long gt = j % p.ntg, gc = (j / p.ntg) % p.cin_groups, gi = j / (p.ntg * p.cin_groups);
    const int t_cnt = (int)((p.taps - gt * p.dt) < p.dt ? (p.taps - gt * p.dt) : p.dt);
    int n = 0;
    for (int r = 0; r < p.dr; ++r)
        for (int c = 0; c < p.dk; ++c)
            for (int t = 0; t < t_cnt; ++t)
                idx[n++] = (gi * p.dr + r) * p.cols + (gc * p.dk + c) * p.taps + gt * p.dt + t;
    return n;
}

__device__ __forceinline__ double tree(double (&t)[16], int n) {
    for (int w = 1; w < n; w <<= 1)
        for (int i = 0; i < n; i += 2 * w) t[i] = __dadd_rn(t[i], t[i + w]);
    return t[0];
}

// S = sum|v|, q = S / n, Lu = sum(|v| - q)^2, sumsq = sum v^2: every operation rounded on its own
__device__ __forceinline__ void keys_of(const float (&v)[16], int n, double *S, double *q, double *Lu, double *sumsq) {
    double a[16], t[16];
    for (int l = 0; l < n; ++l) { a[l] = (double)fabsf(v[l]); t[l] = a[l]; }
    *S = tree(t, n);
    *q = __dmul_rn(*S, 1.0 / (double)n);               // n is a power of two: exact scaling
    for (int l = 0; l < n; ++l) { const double d = __dsub_rn(a[l], *q); t[l] = __dmul_rn(d, d); }
    *Lu = tree(t, n);
    for (int l = 0; l < n; ++l) t[l] = __dmul_rn(a[l], a[l]);
    *sumsq = tree(t, n);
}

__device__ __forceinline__ int load_members(const SParams &p, long long j, long long (&idx)[16], float (&v)[16]) {
    const int n = block_members(p, j, idx);
    for (int l = 0; l < n; ++l) {
        float w = __ldg(p.W + idx[l]);
        if (p.U) w = __fadd_rn(w, __ldg(p.U + idx[l]));
        v[l] = w;
    }
    return n;
}

__global__ void __launch_bounds__(256) shape_stats_kernel(SParams p, double *key_p, double *key_u, double *loss_u,
                                                          double *loss_p, unsigned *dev_status) {
    unsigned bad = 0;
    for (long long j = (long long)blockIdx.x * blockDim.x + threadIdx.x; j < p.mb; j += (long long)gridDim.x * blockDim.x) {
        long long idx[16];
        float v[16];
        const int n = load_members(p, j, idx, v);
        double S, q, Lu, sq;
        keys_of(v, n, &S, &q, &Lu, &sq);
        bad |= ((unsigned)__double2hiint(S) >= 0x7ff00000u) ? 1u : 0u;       // Inf or NaN among the weights
        const double kp = p.use_l1 ? S : sq;
        key_p[j] = kp;
        key_u[j] = Lu;
        if (loss_u) loss_u[j] = Lu;
        if (loss_p) loss_p[j] = kp;
    }
    if (bad) atomicOr(dev_status, (unsigned)MWU_DEV_NONFINITE);
}

__global__ void __launch_bounds__(256) sign_plane_kernel(const float *W, const float *U, long long n, unsigned *sign_bits) {
    const long long n_words = (n + 31) / 32;
    for (long long wi = (long long)blockIdx.x * blockDim.x + threadIdx.x; wi < n_words; wi += (long long)gridDim.x * blockDim.x) {
        unsigned word = 0;
        for (int b = 0; b < 32; ++b) {
            const long long f = wi * 32 + b;
            if (f < n) {
                float w = __ldg(W + f);
                if (U) w = __fadd_rn(w, __ldg(U + f));
                word |= (w < 0.f ? 1u : 0u) << b;
            }
        }
        sign_bits[wi] = word;
    }
}

__device__ __forceinline__ unsigned block_scan_incl(unsigned x, unsigned *s_warp) {
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    for (int m = 1; m < 32; m <<= 1) {
        const unsigned y = __shfl_up_sync(0xffffffffu, x, m);
        if (lane >= m) x += y;
    }
    if (lane == 31) s_warp[w] = x;
    __syncthreads();
    if (w == 0) {
        unsigned t = s_warp[lane];
        for (int m = 1; m < 32; m <<= 1) {
            const unsigned y = __shfl_up_sync(0xffffffffu, t, m);
            if (lane >= m) t += y;
        }
        s_warp[lane] = t;
    }
    __syncthreads();
    const unsigned add = w ? s_warp[w - 1] : 0u;
    __syncthreads();
    return x + add;
}

// One CTA: bit i of `out` is set for the k entries with the smallest (key, index) among the entries
// whose bit in `exclude` is clear (exclude may be null).  Keys are non-negative doubles, compared
// through their bit patterns.  k larger than the eligible count selects all eligible entries.
__global__ void __launch_bounds__(SEL_THREADS) select_smallest_kernel(const double *key, unsigned n, unsigned k,
                                                                      const unsigned *exclude, unsigned *out) {
    __shared__ unsigned s_hist[256];
    __shared__ u64 s_prefix;
    __shared__ unsigned s_r, s_all;
    __shared__ unsigned s_warp[32];
    const u64 *keys = reinterpret_cast<const u64 *>(key);
    const unsigned n_words = (n + 31u) / 32u;
    auto eligible = [&](unsigned i) -> bool { return !exclude || !((exclude[i >> 5] >> (i & 31u)) & 1u); };
    if (threadIdx.x == 0) { s_prefix = 0; s_r = k; s_all = 0; }
    __syncthreads();
    u64 mask = 0;
    if (k > 0u) {
        for (int shift = 56; shift >= 0; shift -= 8) {
            for (unsigned i = threadIdx.x; i < 256u; i += blockDim.x) s_hist[i] = 0;
            __syncthreads();
            const u64 prefix = s_prefix;
            for (unsigned i = threadIdx.x; i < n; i += blockDim.x) {
                const u64 kk = keys[i];
                if ((kk & mask) == prefix && eligible(i)) atomicAdd(&s_hist[(unsigned)(kk >> shift) & 255u], 1u);
            }
            __syncthreads();
            if (threadIdx.x == 0) {
                unsigned r = s_r, d = 0;
                while (d < 256u && s_hist[d] < r) { r -= s_hist[d]; ++d; }
                if (d == 256u) { s_all = 1; d = 255; }  // fewer than k eligible entries under this prefix: take everything
                s_r = r;
                s_prefix = prefix | ((u64)d << shift);
            }
            mask |= (u64)255 << shift;
            __syncthreads();
            if (s_all) break;
        }
    }
    const bool all = s_all != 0u;
    const u64 T = s_prefix;
    const unsigned r_ties = s_r;
    const unsigned words_per = (n_words + blockDim.x - 1u) / blockDim.x;
    const unsigned w0 = threadIdx.x * words_per, w1 = w0 + words_per < n_words ? w0 + words_per : n_words;
    unsigned ties = 0;
    if (k > 0u && !all)
        for (unsigned wi = w0; wi < w1; ++wi)
            for (unsigned bit = 0; bit < 32u; ++bit) {
                const unsigned i = wi * 32u + bit;
                if (i < n && keys[i] == T && eligible(i)) ++ties;
            }
    const unsigned incl = block_scan_incl(ties, s_warp);
    unsigned ordinal = incl - ties;
    for (unsigned wi = w0; wi < w1; ++wi) {
        unsigned wv = 0;
        for (unsigned bit = 0; bit < 32u; ++bit) {
            const unsigned i = wi * 32u + bit;
            if (i >= n) break;
            if (k == 0u || !eligible(i)) continue;
            bool take = all;
            if (!all) {
                const u64 kk = keys[i];
                take = kk < T;
                if (kk == T) { take = ordinal < r_ties; ++ordinal; }
            }
            wv |= (take ? 1u : 0u) << bit;
        }
        out[wi] = wv;
    }
}

__global__ void __launch_bounds__(256) shape_emit_kernel(SParams p, const unsigned *pruned_bitmap,
                                                         const unsigned *unified_bitmap, float *Q, float *u_out,
                                                         float *U_next, double *resid) {
    double acc = 0.0;
    for (long long j = (long long)blockIdx.x * blockDim.x + threadIdx.x; j < p.mb; j += (long long)gridDim.x * blockDim.x) {
        long long idx[16];
        float v[16];
        const int n = load_members(p, j, idx, v);
        const bool pr = (pruned_bitmap[j >> 5] >> (j & 31)) & 1u;
        const bool un = !pr && ((unified_bitmap[j >> 5] >> (j & 31)) & 1u);
        float qf = 0.f;
        if (un || (resid && pr)) {
            double S, q, Lu, sq;
            keys_of(v, n, &S, &q, &Lu, &sq);
            qf = __double2float_rn(q);
            if (resid) acc += pr ? sq : Lu;
        }
        u_out[j] = un ? qf : 0.f;
        for (int l = 0; l < n; ++l) {
            const float q = pr ? 0.f : (un ? (v[l] < 0.f ? -qf : qf) : v[l]);
            if (Q) Q[idx[l]] = q;
            if (U_next) U_next[idx[l]] = __fsub_rn(v[l], q);
        }
    }
    if (resid) {
        for (int m = 16; m > 0; m >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, m);
        if ((threadIdx.x & 31) == 0 && acc != 0.0) atomicAdd(resid, acc);
    }
}

// 1-dim run jb = row * (cols / dk) + kb belongs to block (row / dr, kb): its class and magnitude
__global__ void __launch_bounds__(256) lower_kernel(long long n_runs, long long runs_per_row, int dr,
                                                    const unsigned *pruned_bitmap, const unsigned *unified_bitmap,
                                                    const float *u, unsigned *pruned1, unsigned *unified1, float *u1) {
    const long long n_iter = (n_runs + 31) / 32 * 32;
    for (long long jb = (long long)blockIdx.x * blockDim.x + threadIdx.x; jb < n_iter; jb += (long long)gridDim.x * blockDim.x) {
        bool pr = false, un = false;
        if (jb < n_runs) {
            const long long row = jb / runs_per_row, kb = jb - row * runs_per_row;
            const long long j = (row / dr) * runs_per_row + kb;
            pr = (pruned_bitmap[j >> 5] >> (j & 31)) & 1u;
            un = (unified_bitmap[j >> 5] >> (j & 31)) & 1u;
            u1[jb] = u[j];
        }
        const unsigned wp = __ballot_sync(0xffffffffu, pr), wu = __ballot_sync(0xffffffffu, un);
        if ((threadIdx.x & 31) == 0 && jb < n_runs) { pruned1[jb >> 5] = wp; unified1[jb >> 5] = wu; }
    }
}

static int grid_for(long long items, int sm_count) {
    const long long want = (items + 255) / 256, cap = (long long)sm_count * 16;
    return (int)(want < cap ? (want > 0 ? want : 1) : cap);
}

// bytes of scratch the shape path needs: the two key arrays
size_t workspace_bytes(const mwu_proj_desc *desc) {
    const ShapeInfo sh = shape_of(desc);
    return align_up((size_t)sh.mb * sizeof(double)) * 2 + 256;
}

int project(const mwu_proj_desc *desc, const float *W, const float *U_dual, float *Q, float *U_next,
            double *residual_sq, float *u, uint32_t *pruned_bitmap, uint32_t *unified_bitmap, uint32_t *sign_bits,
            double *loss_u, double *loss_p, uint32_t *dev_status, void *workspace, int sm_count, cudaStream_t st) {
    const ShapeInfo sh = shape_of(desc);
    SParams p;
    p.W = W; p.U = U_dual;
    p.rows = desc->rows; p.cols = desc->cols;
    p.dk = sh.dk; p.dr = sh.dr; p.dt = sh.dt; p.taps = sh.taps;
    p.cin_groups = sh.cin_groups; p.ntg = sh.ntg; p.mb = sh.mb;
    p.use_l1 = desc->prune_key == MWU_PRUNE_KEY_L1;
    double *key_p = (double *)workspace;
    double *key_u = (double *)((char *)workspace + align_up((size_t)sh.mb * sizeof(double)));
    if (residual_sq && cudaMemsetAsync(residual_sq, 0, sizeof(double), st) != cudaSuccess) return MWU_ERR_CUDA;
    shape_stats_kernel<<<grid_for(sh.mb, sm_count), 256, 0, st>>>(p, key_p, key_u, loss_u, loss_p, dev_status);
    const long long n = desc->rows * desc->cols;
    sign_plane_kernel<<<grid_for((n + 31) / 32, sm_count), 256, 0, st>>>(W, U_dual, n, sign_bits);
    select_smallest_kernel<<<1, SEL_THREADS, 0, st>>>(key_p, (unsigned)sh.mb, (unsigned)desc->k_prune, nullptr, pruned_bitmap);
    select_smallest_kernel<<<1, SEL_THREADS, 0, st>>>(key_u, (unsigned)sh.mb, (unsigned)(desc->k_unify - desc->k_prune),
                                                      pruned_bitmap, unified_bitmap);
    shape_emit_kernel<<<grid_for(sh.mb, sm_count), 256, 0, st>>>(p, pruned_bitmap, unified_bitmap, Q, u, U_next, residual_sq);
    count_launch(5);
    return cudaGetLastError() == cudaSuccess ? MWU_OK : MWU_ERR_CUDA;
}

// scratch mwu_pack needs behind the packed bytes for a shaped descriptor: lowered u and bitmaps
size_t lowering_bytes(const mwu_proj_desc *desc) {
    const size_t runs = (size_t)(desc->rows * desc->cols / desc->block);
    return align_up(runs * sizeof(float)) + 2 * align_up((runs + 31) / 32 * 4 + 16);
}

int lower(const mwu_proj_desc *desc, const float *u, const uint32_t *pruned_bitmap, const uint32_t *unified_bitmap,
          void *scratch, const float **u1, const uint32_t **pruned1, const uint32_t **unified1, int sm_count,
          cudaStream_t st) {
    const ShapeInfo sh = shape_of(desc);
    const long long runs = desc->rows * desc->cols / desc->block;
    float *du = (float *)scratch;
    unsigned *dp = (unsigned *)((char *)scratch + align_up((size_t)runs * sizeof(float)));
    unsigned *dun = (unsigned *)((char *)dp + align_up(((size_t)runs + 31) / 32 * 4 + 16));
    lower_kernel<<<grid_for(runs, sm_count), 256, 0, st>>>(runs, desc->cols / desc->block, sh.dr, pruned_bitmap,
                                                          unified_bitmap, u, dp, dun, du);
    count_launch();
    *u1 = du; *pruned1 = dp; *unified1 = dun;
    return cudaGetLastError() == cudaSuccess ? MWU_OK : MWU_ERR_CUDA;
}

}  // namespace shapes
}  // namespace mwu
