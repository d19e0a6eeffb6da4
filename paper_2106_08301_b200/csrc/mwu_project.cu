// mwu_project: Q = Unify(W + U), the Q-step of ADMM (Algorithm 1, Eq. 7) for 1-D micro-blocks.
//
// Pipeline (all on the caller's stream, no host synchronisation):
//   sample_kernel   one CTA looks at <= 4096 evenly spaced blocks and places a narrow window of
//                   8190 bins around the k-th smallest key of each selection (prune key, L_u).
//                   The window only steers efficiency; any window gives the same result.
//   stats_kernel    streams W (+U) once with 128-bit loads; per block the fp64 keys
//                   (Section 3.1: q = mean|v|, L_u = sum(|v|-q)^2, L_p = sum v^2) are reduced with
//                   warp shuffles; writes a 2x16-bit bin code per block and the prune histogram.
//   resolve_kernel  (cooperative, once per selection) finds the exact threshold element
//                   (key, block index): scans the histogram, narrows the range of the composite
//                   96-bit key until <= 2048 candidates remain, sorts them in shared memory.
//   emit_kernel     streams W again: classifies every block from its bin code (exact key only
//                   for blocks in the threshold bin), writes Q, u, both bitmaps, the sign plane.
#include <cooperative_groups.h>

#include "mwu_common.cuh"

namespace cg = cooperative_groups;

namespace mwu {
namespace proj {

constexpr int NB = 8192;        // level-0 bins: 0 = below the window, NB-1 = above it
constexpr int CAP = 2048;       // candidates sorted by the last step
constexpr int NSAMP = 4096;
constexpr int RESOLVE_THREADS = 1024;

typedef unsigned long long u64;
typedef unsigned __int128 u128;

struct Sel {
    u64 lo0, hi0;               // level-0 window on the key's bit pattern
    unsigned shift0;
    unsigned mode;              // 0: threshold, 1: nothing selected, 2: everything eligible selected
    u64 k;                      // how many to select
    unsigned B;                 // level-0 bin that holds the threshold element
    unsigned pad0;
    u64 r;                      // rank (1-based) of the threshold element inside [lo, hi)
    u64 cnt;                    // eligible elements inside [lo, hi)
    u64 lo_hi, lo_lo, hi_hi, hi_lo;   // composite (key << 32 | index) range, as two 64-bit halves
    u64 T_key, T_idx;           // selected  <=>  (key, index) <= (T_key, T_idx)
};

struct Work {
    Sel sel[2];                 // 0: prune, 1: unify
    unsigned cand_count[2];
    unsigned pad[2];
};

struct Params {
    const float *W;
    const float *U;
    long long n_floats;         // rows * cols
    long long n_blocks;
    int b;
    int use_l1;
    Work *work;
    unsigned *hist;             // [3][NB]: prune, unify, refine scratch
    u64 *cand_key;              // [CAP]
    unsigned *cand_idx;         // [CAP]
    unsigned *bins;             // [n_blocks]
    unsigned *dev_status;
};

__device__ __forceinline__ u128 make_c(u64 key, u64 idx) { return ((u128)key << 32) | (u128)idx; }
__device__ __forceinline__ u128 from_halves(u64 hi, u64 lo) { return ((u128)hi << 64) | (u128)lo; }

__device__ __forceinline__ unsigned bin_of(u64 key, u64 lo0, u64 hi0, unsigned shift0) {
    if (key < lo0) return 0u;
    if (key >= hi0) return (unsigned)(NB - 1);
    return 1u + (unsigned)((key - lo0) >> shift0);
}

template <typename T>
__device__ __forceinline__ T ld_vol(const T *p) { return *reinterpret_cast<const volatile T *>(p); }

// ---------------------------------------------------------------------------------------------
// exact keys of one block by one thread (sampling and the rare threshold-bin paths)
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ float load_v(const float *W, const float *U, long long f) {
    float w = __ldg(W + f);
    if (U) w = __fadd_rn(w, __ldg(U + f));
    return w;
}

__device__ __noinline__ void block_keys_scalar(const float *W, const float *U, long long j, int b,
                                               int use_l1, double *S_out, double *Lu_out,
                                               double *Kp_out) {
    double a[16], t[16];
    for (int l = 0; l < b; ++l) a[l] = (double)fabsf(load_v(W, U, j * b + l));
    for (int l = 0; l < b; ++l) t[l] = a[l];
    for (int w = 1; w < b; w <<= 1)
        for (int i = 0; i < b; i += 2 * w) t[i] = __dadd_rn(t[i], t[i + w]);
    const double S = t[0];
    const double q = __dmul_rn(S, 1.0 / (double)b);
    for (int l = 0; l < b; ++l) {
        const double d = __dsub_rn(a[l], q);
        t[l] = __dmul_rn(d, d);
    }
    for (int w = 1; w < b; w <<= 1)
        for (int i = 0; i < b; i += 2 * w) t[i] = __dadd_rn(t[i], t[i + w]);
    *Lu_out = t[0];
    *S_out = S;
    if (use_l1) {
        *Kp_out = S;
    } else {
        for (int l = 0; l < b; ++l) t[l] = __dmul_rn(a[l], a[l]);
        for (int w = 1; w < b; w <<= 1)
            for (int i = 0; i < b; i += 2 * w) t[i] = __dadd_rn(t[i], t[i + w]);
        *Kp_out = t[0];
    }
}

__device__ __forceinline__ u64 key_bits(double x) { return (u64)__double_as_longlong(x); }

// ---------------------------------------------------------------------------------------------
// sample_kernel: choose the level-0 windows
// ---------------------------------------------------------------------------------------------
__device__ void bitonic_sort_u64(u64 *a, int n_pow2) {
    for (int k = 2; k <= n_pow2; k <<= 1) {
        for (int j = k >> 1; j > 0; j >>= 1) {
            for (int i = threadIdx.x; i < n_pow2; i += blockDim.x) {
                const int ixj = i ^ j;
                if (ixj > i) {
                    const u64 x = a[i], y = a[ixj];
                    const bool up = ((i & k) == 0);
                    if ((x > y) == up) { a[i] = y; a[ixj] = x; }
                }
            }
            __syncthreads();
        }
    }
}

__device__ void window_from_sorted(const u64 *a, int n, double frac, Sel *s) {
    // n sorted sample keys; the target quantile is `frac`; keep +-4 sigma (binomial) around it
    const double pos = frac * n;
    const double margin = 4.0 * sqrt(fmax(n * frac * (1.0 - frac), 0.0)) + 4.0;
    long long il = (long long)floor(pos - margin);
    long long ih = (long long)ceil(pos + margin);
    if (il < 0) il = 0;
    if (ih > n - 1) ih = n - 1;
    u64 lo = a[il], hi = a[ih];
    if (hi < lo) hi = lo;
    unsigned shift = 0;
    while (((hi - lo) >> shift) >= (u64)(NB - 2)) ++shift;
    s->lo0 = lo;
    s->hi0 = hi;
    s->shift0 = shift;
}

__global__ void __launch_bounds__(1024) sample_kernel(Params p, long long k_unify, long long k_prune) {
    __shared__ u64 skey[NSAMP];
    __shared__ int s_kept;
    __shared__ u64 s_That;
    const long long mb = p.n_blocks;
    const int ns = (int)(mb < (long long)NSAMP ? mb : (long long)NSAMP);
    const int per = NSAMP / 1024;
    u64 kp[per], ku[per];
    if (threadIdx.x == 0) s_kept = 0;
    for (int t = 0; t < per; ++t) {
        const int i = threadIdx.x + t * 1024;
        kp[t] = ~0ull;
        ku[t] = ~0ull;
        if (i < ns) {
            const long long j = (long long)(((u128)(u64)i * (u128)(u64)mb) / (u128)(u64)ns);
            double S, Lu, Kp;
            block_keys_scalar(p.W, p.U, j, p.b, p.use_l1, &S, &Lu, &Kp);
            kp[t] = key_bits(Kp);
            ku[t] = key_bits(Lu);
        }
        skey[i] = kp[t];
    }
    __syncthreads();
    Sel *sp = &p.work->sel[0];
    Sel *su = &p.work->sel[1];
    const long long ksel_u = k_unify - k_prune;
    bitonic_sort_u64(skey, NSAMP);
    if (threadIdx.x == 0) {
        const double fp = (double)k_prune / (double)mb;
        window_from_sorted(skey, ns, fp, sp);
        sp->mode = (k_prune == 0) ? 1u : (k_prune == mb ? 2u : 0u);
        sp->k = (u64)k_prune;
        long long pos = (long long)(fp * ns);
        if (pos > ns - 1) pos = ns - 1;
        s_That = (k_prune == 0) ? 0ull : skey[pos];
    }
    __syncthreads();
    const u64 That = s_That;
    const bool none_pruned = (k_prune == 0);
    __syncthreads();
    int kept = 0;
    for (int t = 0; t < per; ++t) {
        const int i = threadIdx.x + t * 1024;
        u64 v = ~0ull;
        if (i < ns && (none_pruned || kp[t] > That)) { v = ku[t]; ++kept; }
        skey[i] = v;
    }
    atomicAdd(&s_kept, kept);
    __syncthreads();
    bitonic_sort_u64(skey, NSAMP);
    if (threadIdx.x == 0) {
        const int nr = s_kept > 0 ? s_kept : 1;
        const long long elig = mb - k_prune;
        const double fu = elig > 0 ? (double)ksel_u / (double)elig : 0.0;
        window_from_sorted(skey, nr, fu, su);
        su->mode = (ksel_u == 0) ? 1u : (ksel_u == elig ? 2u : 0u);
        su->k = (u64)ksel_u;
    }
}

// ---------------------------------------------------------------------------------------------
// per-thread / per-group fp64 statistics with the fixed pairwise tree
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ double shfl_xor_f64(double x, int m) {
    return __shfl_xor_sync(0xffffffffu, x, m);
}

// loads 4 consecutive floats starting at f (f % 4 == 0); zero beyond n
__device__ __forceinline__ float4 load4(const float *W, const float *U, long long f, long long n,
                                        bool *nonfinite) {
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (f + 3 < n) {
        v = __ldg(reinterpret_cast<const float4 *>(W + f));
        if (U) {
            const float4 d = __ldg(reinterpret_cast<const float4 *>(U + f));
            v.x = __fadd_rn(v.x, d.x); v.y = __fadd_rn(v.y, d.y);
            v.z = __fadd_rn(v.z, d.z); v.w = __fadd_rn(v.w, d.w);
        }
    } else if (f < n) {
        float t[4] = {0.f, 0.f, 0.f, 0.f};
        for (int l = 0; l < 4 && f + l < n; ++l) t[l] = load_v(W, U, f + l);
        v = make_float4(t[0], t[1], t[2], t[3]);
    }
    const unsigned ex = 0x7f800000u;
    *nonfinite = ((__float_as_uint(v.x) & ex) == ex) | ((__float_as_uint(v.y) & ex) == ex) |
                 ((__float_as_uint(v.z) & ex) == ex) | ((__float_as_uint(v.w) & ex) == ex);
    return v;
}

// Keys of the block(s) a thread touches.  For B >= 8 the block spans B/4 neighbouring lanes.
// On return (B >= 8): every lane of the group holds S; even lanes hold L_u in `first`, odd
// lanes hold the prune key in `first`.  For B == 4: first = L_u, second = prune key.
// For B == 2: handled by keys_b2.
template <int B>
__device__ __forceinline__ void keys_group(const float4 v, int use_l1, double *S_out, double *first,
                                           double *second) {
    const double a0 = (double)fabsf(v.x), a1 = (double)fabsf(v.y);
    const double a2 = (double)fabsf(v.z), a3 = (double)fabsf(v.w);
    double S = __dadd_rn(__dadd_rn(a0, a1), __dadd_rn(a2, a3));
    if (B >= 8) S = __dadd_rn(S, shfl_xor_f64(S, 1));
    if (B >= 16) S = __dadd_rn(S, shfl_xor_f64(S, 2));
    const double q = __dmul_rn(S, 1.0 / (double)B);
    const double d0 = __dsub_rn(a0, q), d1 = __dsub_rn(a1, q);
    const double d2 = __dsub_rn(a2, q), d3 = __dsub_rn(a3, q);
    double Lu = __dadd_rn(__dadd_rn(__dmul_rn(d0, d0), __dmul_rn(d1, d1)),
                          __dadd_rn(__dmul_rn(d2, d2), __dmul_rn(d3, d3)));
    double Kp;
    if (use_l1) {
        Kp = 0.0;   // replaced by S below
    } else {
        // a*a is exact in fp64 for fp32-valued a, so fma(a,a,c) == round(a*a + c): same bits
        // as a separately rounded multiply and add.
        Kp = __dadd_rn(__fma_rn(a0, a0, __dmul_rn(a1, a1)), __fma_rn(a2, a2, __dmul_rn(a3, a3)));
    }
    if (B >= 8) {
        const bool odd = (threadIdx.x & 1) != 0;
        const double send = odd ? Lu : Kp;
        const double keep = odd ? Kp : Lu;
        double res = __dadd_rn(keep, shfl_xor_f64(send, 1));
        if (B >= 16) res = __dadd_rn(res, shfl_xor_f64(res, 2));
        if (use_l1 && odd) res = S;
        *first = res;
        *second = 0.0;
    } else {
        *first = Lu;
        *second = use_l1 ? S : Kp;
    }
    *S_out = S;
}

__device__ __forceinline__ void keys_b2(float x, float y, int use_l1, double *S_out, double *Lu,
                                        double *Kp) {
    const double a0 = (double)fabsf(x), a1 = (double)fabsf(y);
    const double S = __dadd_rn(a0, a1);
    const double q = __dmul_rn(S, 0.5);
    const double d0 = __dsub_rn(a0, q), d1 = __dsub_rn(a1, q);
    *Lu = __dadd_rn(__dmul_rn(d0, d0), __dmul_rn(d1, d1));
    *Kp = use_l1 ? S : __fma_rn(a0, a0, __dmul_rn(a1, a1));
    *S_out = S;
}

// ---------------------------------------------------------------------------------------------
// stats_kernel
// ---------------------------------------------------------------------------------------------
template <int B>
__global__ void __launch_bounds__(256) stats_kernel(Params p, double *loss_u, double *loss_p) {
    const Sel *sp = &p.work->sel[0];
    const Sel *su = &p.work->sel[1];
    const u64 plo = sp->lo0, phi = sp->hi0, ulo = su->lo0, uhi = su->hi0;
    const unsigned psh = sp->shift0, ush = su->shift0;
    unsigned cnt_under = 0, cnt_over = 0;
    bool any_nonfinite = false;
    const long long n = p.n_floats;
    const long long n_quads = (n + 3) / 4;
    // a warp always walks whole groups of 32 quads so that shuffles see all lanes
    const long long n_iter = (n_quads + 31) / 32 * 32;
    for (long long qd = (long long)blockIdx.x * blockDim.x + threadIdx.x; qd < n_iter;
         qd += (long long)gridDim.x * blockDim.x) {
        const long long f = qd * 4;
        bool nf;
        const float4 v = load4(p.W, p.U, f, n, &nf);
        any_nonfinite |= nf;
        if (B == 2) {
            double S, Lu, Kp;
            unsigned code[2];
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                keys_b2(e ? v.z : v.x, e ? v.w : v.y, p.use_l1, &S, &Lu, &Kp);
                const long long j = f / 2 + e;
                const unsigned bu = bin_of(key_bits(Lu), ulo, uhi, ush);
                const unsigned bp = bin_of(key_bits(Kp), plo, phi, psh);
                code[e] = bp | (bu << 16);
                if (j < p.n_blocks) {
                    if (bp == 0) ++cnt_under;
                    else if (bp == NB - 1) ++cnt_over;
                    else atomicAdd(&p.hist[bp], 1u);
                    if (loss_u) loss_u[j] = Lu;
                    if (loss_p) loss_p[j] = Kp;
                }
            }
            const long long j0 = f / 2;
            if (j0 + 1 < p.n_blocks) {
                *reinterpret_cast<uint2 *>(p.bins + j0) = make_uint2(code[0], code[1]);
            } else if (j0 < p.n_blocks) {
                p.bins[j0] = code[0];
            }
        } else {
            constexpr int LPB = (B >= 4) ? B / 4 : 1;      // lanes per block
            double S, first, second;
            keys_group<B>(v, p.use_l1, &S, &first, &second);
            const long long j = f / B;
            if (B == 4) {
                const unsigned bu = bin_of(key_bits(first), ulo, uhi, ush);
                const unsigned bp = bin_of(key_bits(second), plo, phi, psh);
                if (j < p.n_blocks) {
                    p.bins[j] = bp | (bu << 16);
                    if (bp == 0) ++cnt_under;
                    else if (bp == NB - 1) ++cnt_over;
                    else atomicAdd(&p.hist[bp], 1u);
                    if (loss_u) loss_u[j] = first;
                    if (loss_p) loss_p[j] = second;
                }
            } else {
                const bool odd = (threadIdx.x & 1) != 0;
                const unsigned mine = odd ? bin_of(key_bits(first), plo, phi, psh)
                                          : (bin_of(key_bits(first), ulo, uhi, ush) << 16);
                const unsigned code = mine | __shfl_xor_sync(0xffffffffu, mine, 1);
                const int sub = threadIdx.x & (LPB - 1);
                if (j < p.n_blocks) {
                    if (sub == 0) {
                        p.bins[j] = code;
                        if (loss_u) loss_u[j] = first;
                    } else if (sub == 1) {
                        const unsigned bp = mine;
                        if (bp == 0) ++cnt_under;
                        else if (bp == NB - 1) ++cnt_over;
                        else atomicAdd(&p.hist[bp], 1u);
                        if (loss_p) loss_p[j] = first;
                    }
                }
            }
        }
    }
    // block-level totals of the two catch-all bins
    __shared__ unsigned s_under, s_over;
    if (threadIdx.x == 0) { s_under = 0; s_over = 0; }
    __syncthreads();
    for (int m = 16; m > 0; m >>= 1) {
        cnt_under += __shfl_xor_sync(0xffffffffu, cnt_under, m);
        cnt_over += __shfl_xor_sync(0xffffffffu, cnt_over, m);
    }
    if ((threadIdx.x & 31) == 0) {
        if (cnt_under) atomicAdd(&s_under, cnt_under);
        if (cnt_over) atomicAdd(&s_over, cnt_over);
    }
    if (any_nonfinite) atomicOr(p.dev_status, (unsigned)MWU_DEV_NONFINITE);
    __syncthreads();
    if (threadIdx.x == 0) {
        if (s_under) atomicAdd(&p.hist[0], s_under);
        if (s_over) atomicAdd(&p.hist[NB - 1], s_over);
    }
}

// ---------------------------------------------------------------------------------------------
// classification helpers shared by resolve and emit
// ---------------------------------------------------------------------------------------------
struct SelView {            // read-only copy of what classification needs
    unsigned mode, B;
    u64 T_key, T_idx;
};

__device__ __forceinline__ SelView view_of(const Sel *s) {
    SelView v;
    v.mode = ld_vol(&s->mode);
    v.B = ld_vol(&s->B);
    v.T_key = ld_vol(&s->T_key);
    v.T_idx = ld_vol(&s->T_idx);
    return v;
}

// which: 0 -> prune key, 1 -> L_u
__device__ __forceinline__ u64 exact_key(const Params &p, long long j, int which) {
    double S, Lu, Kp;
    block_keys_scalar(p.W, p.U, j, p.b, p.use_l1, &S, &Lu, &Kp);
    return key_bits(which ? Lu : Kp);
}

__device__ __forceinline__ bool selected(const Params &p, const SelView &s, long long j,
                                         unsigned bin, int which) {
    if (s.mode == 1u) return false;
    if (s.mode == 2u) return true;
    if (bin < s.B) return true;
    if (bin > s.B) return false;
    const u64 key = exact_key(p, j, which);
    return key < s.T_key || (key == s.T_key && (u64)j <= s.T_idx);
}

// ---------------------------------------------------------------------------------------------
// resolve_kernel: exact threshold element of one selection
// ---------------------------------------------------------------------------------------------
// block 0: find the bin holding the r-th element; hist has NB entries
__device__ void scan_hist(const unsigned *hist, u64 r, unsigned *bin_out, u64 *r_in_bin,
                          u64 *cnt_out, unsigned *err) {
    __shared__ u64 s_part[RESOLVE_THREADS];
    constexpr int PER = NB / RESOLVE_THREADS;
    u64 local[PER];
    u64 sum = 0;
    for (int i = 0; i < PER; ++i) {
        local[i] = ld_vol(&hist[threadIdx.x * PER + i]);
        sum += local[i];
    }
    s_part[threadIdx.x] = sum;
    __syncthreads();
    // inclusive scan (Hillis-Steele), 1024 entries
    for (int off = 1; off < RESOLVE_THREADS; off <<= 1) {
        u64 add = 0;
        if ((int)threadIdx.x >= off) add = s_part[threadIdx.x - off];
        __syncthreads();
        s_part[threadIdx.x] += add;
        __syncthreads();
    }
    const u64 incl = s_part[threadIdx.x];
    u64 run = incl - sum;           // exclusive prefix
    if (threadIdx.x == RESOLVE_THREADS - 1 && incl < r) *err = 1;
    for (int i = 0; i < PER; ++i) {
        if (run < r && r <= run + local[i]) {
            *bin_out = threadIdx.x * PER + i;
            *r_in_bin = r - run;
            *cnt_out = local[i];
        }
        run += local[i];
    }
    __syncthreads();
}

__device__ void sort_candidates(u64 *key, unsigned *idx, int n_pow2) {
    for (int k = 2; k <= n_pow2; k <<= 1) {
        for (int j = k >> 1; j > 0; j >>= 1) {
            for (int i = threadIdx.x; i < n_pow2; i += blockDim.x) {
                const int ixj = i ^ j;
                if (ixj > i) {
                    const u64 kx = key[i], ky = key[ixj];
                    const unsigned ix = idx[i], iy = idx[ixj];
                    const bool gt = (kx > ky) || (kx == ky && ix > iy);
                    const bool up = ((i & k) == 0);
                    if (gt == up) { key[i] = ky; key[ixj] = kx; idx[i] = iy; idx[ixj] = ix; }
                }
            }
            __syncthreads();
        }
    }
}

template <int KIND>
__global__ void __launch_bounds__(RESOLVE_THREADS) resolve_kernel(Params p) {
    cg::grid_group grid = cg::this_grid();
    Sel *s = &p.work->sel[KIND];
    unsigned *hist = p.hist + (size_t)KIND * NB;
    unsigned *rhist = p.hist + (size_t)2 * NB;
    const long long stride = (long long)gridDim.x * blockDim.x;
    const long long tid0 = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    __shared__ unsigned s_bin, s_err;
    __shared__ u64 s_r, s_cnt;
    __shared__ u64 c_key[CAP];
    __shared__ unsigned c_idx[CAP];

    SelView prune_view;
    if (KIND == 1) {
        // histogram of L_u over the blocks that were not pruned
        prune_view = view_of(&p.work->sel[0]);
        unsigned under = 0, over = 0;
        for (long long j = tid0; j < p.n_blocks; j += stride) {
            const unsigned code = p.bins[j];
            if (selected(p, prune_view, j, code & 0xffffu, 0)) continue;
            const unsigned bu = code >> 16;
            if (bu == 0) ++under;
            else if (bu == NB - 1) ++over;
            else atomicAdd(&hist[bu], 1u);
        }
        for (int m = 16; m > 0; m >>= 1) {
            under += __shfl_xor_sync(0xffffffffu, under, m);
            over += __shfl_xor_sync(0xffffffffu, over, m);
        }
        if ((threadIdx.x & 31) == 0) {
            if (under) atomicAdd(&hist[0], under);
            if (over) atomicAdd(&hist[NB - 1], over);
        }
        grid.sync();
    }

    // level 0: which bin holds the k-th element
    if (blockIdx.x == 0) {
        if (threadIdx.x == 0) { s_err = 0; s_bin = 0; s_r = 0; s_cnt = 0; }
        __syncthreads();
        scan_hist(hist, s->k, &s_bin, &s_r, &s_cnt, &s_err);
        if (threadIdx.x == 0) {
            if (s_err) atomicOr(p.dev_status, (unsigned)MWU_DEV_SELECT);
            const unsigned B = s_bin;
            u64 klo, khi;      // key range of the bin
            if (B == 0) { klo = 0; khi = s->lo0; }
            else if (B == NB - 1) { klo = s->hi0; khi = ~0ull >> 1; }     // keys are < 2^63
            else {
                klo = s->lo0 + ((u64)(B - 1) << s->shift0);
                khi = s->lo0 + ((u64)B << s->shift0);
                if (khi > s->hi0) khi = s->hi0;
            }
            const u128 lo = make_c(klo, 0), hi = make_c(khi, 0);
            s->B = B;
            s->r = s_r;
            s->cnt = s_cnt;
            s->lo_hi = (u64)(lo >> 64); s->lo_lo = (u64)lo;
            s->hi_hi = (u64)(hi >> 64); s->hi_lo = (u64)hi;
        }
    }
    grid.sync();

    // narrow [lo, hi) until the candidates fit the final sort (normally zero iterations)
    for (int level = 0; level < 10; ++level) {
        if (ld_vol(&s->cnt) <= (u64)CAP) break;
        for (long long i = tid0; i < NB; i += stride) rhist[i] = 0;
        grid.sync();
        const unsigned B = ld_vol(&s->B);
        const u128 lo = from_halves(ld_vol(&s->lo_hi), ld_vol(&s->lo_lo));
        const u128 hi = from_halves(ld_vol(&s->hi_hi), ld_vol(&s->hi_lo));
        unsigned shift = 0;
        while (((hi - lo - 1) >> shift) >= (u128)NB) ++shift;
        for (long long j = tid0; j < p.n_blocks; j += stride) {
            const unsigned code = p.bins[j];
            const unsigned bin = KIND ? (code >> 16) : (code & 0xffffu);
            if (bin != B) continue;
            if (KIND == 1 && selected(p, prune_view, j, code & 0xffffu, 0)) continue;
            const u128 c = make_c(exact_key(p, j, KIND), (u64)j);
            if (c >= lo && c < hi) atomicAdd(&rhist[(unsigned)((c - lo) >> shift)], 1u);
        }
        grid.sync();
        if (blockIdx.x == 0) {
            if (threadIdx.x == 0) s_err = 0;
            __syncthreads();
            scan_hist(rhist, ld_vol(&s->r), &s_bin, &s_r, &s_cnt, &s_err);
            if (threadIdx.x == 0) {
                if (s_err) atomicOr(p.dev_status, (unsigned)MWU_DEV_SELECT);
                u128 nlo = lo + ((u128)s_bin << shift);
                u128 nhi = nlo + ((u128)1 << shift);
                if (nhi > hi) nhi = hi;
                s->r = s_r;
                s->cnt = s_cnt;
                s->lo_hi = (u64)(nlo >> 64); s->lo_lo = (u64)nlo;
                s->hi_hi = (u64)(nhi >> 64); s->hi_lo = (u64)nhi;
            }
        }
        grid.sync();
    }

    // collect the candidates
    {
        const unsigned B = ld_vol(&s->B);
        const u128 lo = from_halves(ld_vol(&s->lo_hi), ld_vol(&s->lo_lo));
        const u128 hi = from_halves(ld_vol(&s->hi_hi), ld_vol(&s->hi_lo));
        for (long long j = tid0; j < p.n_blocks; j += stride) {
            const unsigned code = p.bins[j];
            const unsigned bin = KIND ? (code >> 16) : (code & 0xffffu);
            if (bin != B) continue;
            if (KIND == 1 && selected(p, prune_view, j, code & 0xffffu, 0)) continue;
            const u64 key = exact_key(p, j, KIND);
            const u128 c = make_c(key, (u64)j);
            if (c >= lo && c < hi) {
                const unsigned slot = atomicAdd(&p.work->cand_count[KIND], 1u);
                if (slot < (unsigned)CAP) { p.cand_key[slot] = key; p.cand_idx[slot] = (unsigned)j; }
            }
        }
    }
    grid.sync();

    if (blockIdx.x == 0) {
        const unsigned n = ld_vol(&p.work->cand_count[KIND]);
        const u64 r = ld_vol(&s->r);
        const unsigned m = n < (unsigned)CAP ? n : (unsigned)CAP;
        for (int i = threadIdx.x; i < CAP; i += blockDim.x) {
            c_key[i] = (i < (int)m) ? ld_vol(&p.cand_key[i]) : ~0ull;
            c_idx[i] = (i < (int)m) ? ld_vol(&p.cand_idx[i]) : ~0u;
        }
        __syncthreads();
        sort_candidates(c_key, c_idx, CAP);
        if (threadIdx.x == 0) {
            if (n > (unsigned)CAP || r == 0 || r > (u64)m) {
                atomicOr(p.dev_status, (unsigned)MWU_DEV_SELECT);
                s->T_key = 0; s->T_idx = 0;
            } else {
                s->T_key = c_key[r - 1];
                s->T_idx = (u64)c_idx[r - 1];
            }
        }
    }
}

// ---------------------------------------------------------------------------------------------
// emit_kernel
// ---------------------------------------------------------------------------------------------
template <int B>
__global__ void __launch_bounds__(256) emit_kernel(Params p, float *Q, float *u_out,
                                                   unsigned *pruned_bitmap, unsigned *unified_bitmap,
                                                   unsigned *sign_bits) {
    const SelView vp = view_of(&p.work->sel[0]);
    const SelView vu = view_of(&p.work->sel[1]);
    const long long n = p.n_floats;
    const int lane = threadIdx.x & 31;
    constexpr int CPT = (B >= 4) ? B / 4 : 1;                // 128-float chunks per warp task
    constexpr int BPC = 128 / B;                             // blocks per chunk
    const long long n_chunks = (n + 127) / 128;
    const long long n_tasks = (n_chunks + CPT - 1) / CPT;
    const long long warp0 = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const long long n_warps = ((long long)gridDim.x * blockDim.x) >> 5;
    const long long n_sign_words = (n + 31) / 32;
    const long long n_bm_words = (p.n_blocks + 31) / 32;

    for (long long task = warp0; task < n_tasks; task += n_warps) {
        unsigned word_p = 0, word_u = 0, word_p2 = 0, word_u2 = 0;
#pragma unroll
        for (int it = 0; it < CPT; ++it) {
            const long long chunk = task * CPT + it;
            const long long f = chunk * 128 + lane * 4;
            bool nf;
            const float4 v = load4(p.W, p.U, f, n, &nf);
            float4 q4 = v;
            unsigned cls = 0;           // bit0 pruned, bit1 unified (B == 2: bits 2,3 second block)
            if (B == 2) {
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const long long j = f / 2 + e;
                    const float x = e ? v.z : v.x, y = e ? v.w : v.y;
                    if (j < p.n_blocks) {
                        const unsigned code = p.bins[j];
                        const bool pr = selected(p, vp, j, code & 0xffffu, 0);
                        const bool un = !pr && selected(p, vu, j, code >> 16, 1);
                        float qq = 0.f;
                        if (un) {
                            const double S = __dadd_rn((double)fabsf(x), (double)fabsf(y));
                            qq = __double2float_rn(__dmul_rn(S, 0.5));
                        }
                        float ox = x, oy = y;
                        if (pr) { ox = 0.f; oy = 0.f; }
                        if (un) { ox = (x >= 0.f) ? qq : -qq; oy = (y >= 0.f) ? qq : -qq; }
                        if (e) { q4.z = ox; q4.w = oy; } else { q4.x = ox; q4.y = oy; }
                        u_out[j] = qq;
                        cls |= ((pr ? 1u : 0u) | (un ? 2u : 0u)) << (2 * e);
                    }
                }
            } else {
                constexpr int LPB = B / 4;
                const long long j = f / B;
                const double a0 = (double)fabsf(v.x), a1 = (double)fabsf(v.y);
                const double a2 = (double)fabsf(v.z), a3 = (double)fabsf(v.w);
                double S = __dadd_rn(__dadd_rn(a0, a1), __dadd_rn(a2, a3));
                if (B >= 8) S = __dadd_rn(S, shfl_xor_f64(S, 1));
                if (B >= 16) S = __dadd_rn(S, shfl_xor_f64(S, 2));
                if (j < p.n_blocks) {
                    const unsigned code = p.bins[j];
                    const bool pr = selected(p, vp, j, code & 0xffffu, 0);
                    const bool un = !pr && selected(p, vu, j, code >> 16, 1);
                    float qq = 0.f;
                    if (un) qq = __double2float_rn(__dmul_rn(S, 1.0 / (double)B));
                    if (pr) q4 = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (un) {
                        q4.x = (v.x >= 0.f) ? qq : -qq; q4.y = (v.y >= 0.f) ? qq : -qq;
                        q4.z = (v.z >= 0.f) ? qq : -qq; q4.w = (v.w >= 0.f) ? qq : -qq;
                    }
                    if ((lane & (LPB - 1)) == 0) u_out[j] = qq;
                    cls = (pr ? 1u : 0u) | (un ? 2u : 0u);
                }
            }
            // Q
            if (Q) {
                if (f + 3 < n) {
                    *reinterpret_cast<float4 *>(Q + f) = q4;
                } else if (f < n) {
                    const float t[4] = {q4.x, q4.y, q4.z, q4.w};
                    for (int l = 0; l < 4 && f + l < n; ++l) Q[f + l] = t[l];
                }
            }
            // sign plane: 8 lanes make one 32-bit word
            {
                unsigned nib = (v.x < 0.f ? 1u : 0u) | (v.y < 0.f ? 2u : 0u) |
                               (v.z < 0.f ? 4u : 0u) | (v.w < 0.f ? 8u : 0u);
                nib <<= 4 * (lane & 7);
                nib |= __shfl_xor_sync(0xffffffffu, nib, 1);
                nib |= __shfl_xor_sync(0xffffffffu, nib, 2);
                nib |= __shfl_xor_sync(0xffffffffu, nib, 4);
                const long long wi = chunk * 4 + (lane >> 3);
                if ((lane & 7) == 0 && wi < n_sign_words) sign_bits[wi] = nib;
            }
            // class bitmaps
            if (B == 2) {
                const unsigned c0 = __shfl_sync(0xffffffffu, cls, lane >> 1);
                const unsigned c1 = __shfl_sync(0xffffffffu, cls, 16 + (lane >> 1));
                const unsigned sh = 2 * (lane & 1);
                word_p = __ballot_sync(0xffffffffu, (c0 >> sh) & 1u);
                word_u = __ballot_sync(0xffffffffu, (c0 >> (sh + 1)) & 1u);
                word_p2 = __ballot_sync(0xffffffffu, (c1 >> sh) & 1u);
                word_u2 = __ballot_sync(0xffffffffu, (c1 >> (sh + 1)) & 1u);
            } else {
                constexpr int LPB = B / 4;
                const unsigned c = __shfl_sync(0xffffffffu, cls, (lane * LPB) & 31);
                const unsigned valid = (BPC >= 32) ? 0xffffffffu : ((1u << BPC) - 1u);
                const unsigned bp = __ballot_sync(0xffffffffu, c & 1u) & valid;
                const unsigned bu = __ballot_sync(0xffffffffu, (c >> 1) & 1u) & valid;
                word_p |= bp << ((it * BPC) & 31);
                word_u |= bu << ((it * BPC) & 31);
            }
        }
        if (lane == 0) {
            if (B == 2) {
                const long long w0 = task * 2;
                if (w0 < n_bm_words) { pruned_bitmap[w0] = word_p; unified_bitmap[w0] = word_u; }
                if (w0 + 1 < n_bm_words) { pruned_bitmap[w0 + 1] = word_p2; unified_bitmap[w0 + 1] = word_u2; }
            } else {
                if (task < n_bm_words) { pruned_bitmap[task] = word_p; unified_bitmap[task] = word_u; }
            }
        }
    }
}

}  // namespace proj

// ---------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------
static size_t ws_off_hist() { return align_up(sizeof(proj::Work)); }
static size_t ws_off_cand_key() { return align_up(ws_off_hist() + 3 * proj::NB * sizeof(unsigned)); }
static size_t ws_off_cand_idx() { return align_up(ws_off_cand_key() + proj::CAP * sizeof(proj::u64)); }
static size_t ws_off_bins() { return align_up(ws_off_cand_idx() + proj::CAP * sizeof(unsigned)); }

}  // namespace mwu

extern "C" size_t mwu_project_workspace_bytes(const mwu_proj_desc *desc) {
    if (mwu::validate_desc(desc, false) != MWU_OK) return 0;
    const size_t mb = (size_t)(desc->rows * desc->cols / desc->block);
    return mwu::align_up(mwu::ws_off_bins() + (mb + 8) * sizeof(unsigned));
}

template <int B>
static cudaError_t launch_project(const mwu::proj::Params &p, const mwu_proj_desc *desc, float *Q,
                                  float *u, unsigned *pb, unsigned *ub, unsigned *sb, double *loss_u,
                                  double *loss_p, int sm_count, cudaStream_t st) {
    using namespace mwu::proj;
    const long long n_quads = (p.n_floats + 3) / 4;
    long long want = (n_quads + 255) / 256;
    const long long cap_blocks = (long long)sm_count * 8;
    const int grid_stats = (int)(want < cap_blocks ? (want > 0 ? want : 1) : cap_blocks);
    stats_kernel<B><<<grid_stats, 256, 0, st>>>(p, loss_u, loss_p);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;

    Params pp = p;
    void *args[] = {&pp};
    const long long mb = p.n_blocks;
    long long rb = (mb + RESOLVE_THREADS - 1) / RESOLVE_THREADS;
    const int grid_res = (int)(rb < sm_count ? (rb > 0 ? rb : 1) : sm_count);
    const bool need_p = desc->k_prune > 0 && desc->k_prune < mb;
    const long long ksel_u = desc->k_unify - desc->k_prune;
    const bool need_u = ksel_u > 0 && ksel_u < mb - desc->k_prune;
    if (need_p) {
        e = cudaLaunchCooperativeKernel((void *)resolve_kernel<0>, dim3(grid_res), dim3(RESOLVE_THREADS),
                                        args, 0, st);
        if (e != cudaSuccess) return e;
    }
    if (need_u) {
        e = cudaLaunchCooperativeKernel((void *)resolve_kernel<1>, dim3(grid_res), dim3(RESOLVE_THREADS),
                                        args, 0, st);
        if (e != cudaSuccess) return e;
    }
    constexpr int CPT = (B >= 4) ? B / 4 : 1;
    const long long n_tasks = ((p.n_floats + 127) / 128 + CPT - 1) / CPT;
    long long eb = (n_tasks + 7) / 8;
    const int grid_emit = (int)(eb < cap_blocks ? (eb > 0 ? eb : 1) : cap_blocks);
    emit_kernel<B><<<grid_emit, 256, 0, st>>>(p, Q, u, pb, ub, sb);
    return cudaGetLastError();
}

extern "C" int mwu_project(const mwu_proj_desc *desc, const float *W, const float *U_dual, float *Q,
                           float *u, uint32_t *pruned_bitmap, uint32_t *unified_bitmap,
                           uint32_t *sign_bits, double *loss_u, double *loss_p, uint32_t *dev_status,
                           void *workspace, size_t workspace_bytes, void *cuda_stream) {
    using namespace mwu;
    int rc = validate_desc(desc, false);
    if (rc != MWU_OK) return rc;
    if (!W || !u || !pruned_bitmap || !unified_bitmap || !sign_bits || !dev_status || !workspace)
        return MWU_ERR_INVALID_ARG;
    if (!aligned_to(W, 16) || !aligned_to(U_dual, 16) || !aligned_to(Q, 16) || !aligned_to(u, 16) ||
        !aligned_to(pruned_bitmap, 16) || !aligned_to(unified_bitmap, 16) ||
        !aligned_to(sign_bits, 16) || !aligned_to(loss_u, 16) || !aligned_to(loss_p, 16) ||
        !aligned_to(dev_status, 4) || !aligned_to(workspace, 256))
        return MWU_ERR_ALIGNMENT;
    if (workspace_bytes < mwu_project_workspace_bytes(desc)) return MWU_ERR_WORKSPACE;
    int sm_count = 0;
    rc = check_device(&sm_count);
    if (rc != MWU_OK) return rc;

    cudaStream_t st = (cudaStream_t)cuda_stream;
    char *ws = (char *)workspace;
    proj::Params p;
    p.W = W;
    p.U = U_dual;
    p.n_floats = desc->rows * desc->cols;
    p.n_blocks = p.n_floats / desc->block;
    p.b = desc->block;
    p.use_l1 = desc->prune_key == MWU_PRUNE_KEY_L1;
    p.work = (proj::Work *)ws;
    p.hist = (unsigned *)(ws + ws_off_hist());
    p.cand_key = (proj::u64 *)(ws + ws_off_cand_key());
    p.cand_idx = (unsigned *)(ws + ws_off_cand_idx());
    p.bins = (unsigned *)(ws + ws_off_bins());
    p.dev_status = dev_status;

    if (cudaMemsetAsync(ws, 0, ws_off_cand_key(), st) != cudaSuccess) return MWU_ERR_CUDA;
    proj::sample_kernel<<<1, 1024, 0, st>>>(p, desc->k_unify, desc->k_prune);
    if (cudaGetLastError() != cudaSuccess) return MWU_ERR_CUDA;
    cudaError_t e;
    switch (desc->block) {
        case 2: e = launch_project<2>(p, desc, Q, u, pruned_bitmap, unified_bitmap, sign_bits, loss_u, loss_p, sm_count, st); break;
        case 4: e = launch_project<4>(p, desc, Q, u, pruned_bitmap, unified_bitmap, sign_bits, loss_u, loss_p, sm_count, st); break;
        case 8: e = launch_project<8>(p, desc, Q, u, pruned_bitmap, unified_bitmap, sign_bits, loss_u, loss_p, sm_count, st); break;
        default: e = launch_project<16>(p, desc, Q, u, pruned_bitmap, unified_bitmap, sign_bits, loss_u, loss_p, sm_count, st); break;
    }
    return e == cudaSuccess ? MWU_OK : MWU_ERR_CUDA;
}
