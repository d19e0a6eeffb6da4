// mwu_project: Q = Unify(W + U), the Q-step of ADMM (Algorithm 1, Eq. 7) for 1-D micro-blocks.
//
// Pipeline (all on the caller's stream, no host synchronisation):
//   sample_kernel   one CTA ranks <= 256 evenly spaced blocks and places a narrow window of
//                   8190 bins (65534 above 8M blocks) around the k-th smallest key of each selection (prune key, L_u).
//                   The window only steers efficiency; any window gives the same result.
//   stats_kernel    streams W (+U) once; every thread owns 64 contiguous bytes (four 128-bit
//                   loads in flight) and evaluates the fp64 keys of its blocks (Section 3.1:
//                   q = mean|v|, L_u = sum(|v|-q)^2, L_p = sum v^2) with the fixed pairwise
//                   tree; writes a 2x16-bit bin code per block, the prune-key histogram, the
//                   sign plane and q of every block (into u).
//   prune_select_kernel  locates the bin of the k_prune-th key, then one pass over the bin codes:
//                   blocks of that bin become candidates (normally a few dozen to a few hundred),
//                   blocks above it are counted in the L_u histogram.  The last CTA sorts the
//                   candidates: the result is the exact threshold element (key, block index); it
//                   adds the surviving candidates to the L_u histogram and locates the bin of the
//                   unify threshold.
//   collect_kernel  gathers the blocks of that bin that were not pruned; the last CTA sorts them.
//   emit_kernel     classifies every block from its bin code (exact key only for blocks in a
//                   threshold bin), writes Q, both bitmaps and the final u (0 unless unified).  W
//                   is read again only for the 64-byte units that hold a block keeping its values:
//                   unified blocks are rebuilt from q and the sign plane, pruned ones are zeros.
// When a threshold bin holds more than 2048 blocks (massive ties, e.g. re-projecting an already
// projected tensor) the last CTA narrows the range of the 96-bit composite key (key, index) by
// itself, pass by pass, until the candidates fit: slow but exact.
#include "mwu_common.cuh"

namespace mwu {
namespace proj {

constexpr int NB_MAX = 65536;   // level-0 bins (codes fit 16 bits): bin 0 = below the window, nb-1 = above it
constexpr int NB_SMALL = 8192;  // used up to 8M blocks: fewer bins to clear and scan
constexpr int CAP = 2048;       // candidates sorted by the last step
constexpr int NSAMP = 256;
constexpr int PASS_LOADS = 4;      // 16-byte loads of bin codes a thread keeps in flight in the selection passes
constexpr int FIN_THREADS = 1024;   // block size of the kernels whose last CTA finalises

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
    unsigned ticket[4];         // [1]: prune_select, [3]: collect<1>
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
    int nb;                     // level-0 bins in use (NB_SMALL or NB_MAX)
    unsigned *hist;             // [3][nb]: prune, unify, refine scratch
    u64 *cand_key;              // [CAP]
    unsigned *cand_idx;         // [CAP]
    unsigned *bins;             // [n_blocks]
    unsigned *dev_status;
};

__device__ __forceinline__ u128 make_c(u64 key, u64 idx) { return ((u128)key << 32) | (u128)idx; }
__device__ __forceinline__ u128 from_halves(u64 hi, u64 lo) { return ((u128)hi << 64) | (u128)lo; }

__device__ __forceinline__ unsigned bin_of(u64 key, u64 lo0, u64 hi0, unsigned shift0, unsigned nb) {
    if (key < lo0) return 0u;
    if (key >= hi0) return nb - 1u;
    return 1u + (unsigned)((key - lo0) >> shift0);
}

template <typename T>
__device__ __forceinline__ T ld_vol(const T *p) { return *reinterpret_cast<const volatile T *>(p); }

__device__ __forceinline__ u64 key_bits(double x) { return (u64)__double_as_longlong(x); }

// ---------------------------------------------------------------------------------------------
// fp64 statistics of one block held in registers (fixed pairwise tree, every op rounded alone)
// ---------------------------------------------------------------------------------------------
template <int B>
__device__ __forceinline__ double tree_sum(const double (&x)[B]) {
    double t[B];
#pragma unroll
    for (int l = 0; l < B; ++l) t[l] = x[l];
#pragma unroll
    for (int w = 1; w < B; w <<= 1)
#pragma unroll
        for (int i = 0; i < B; i += 2 * w) t[i] = __dadd_rn(t[i], t[i + w]);
    return t[0];
}

// v: the block's B values.  S = sum|v|, Lu = sum(|v| - S/B)^2, Kp = sum v^2 (or S for the L1 key)
template <int B>
__device__ __forceinline__ void block_keys(const float *v, int use_l1, double *S_out, double *Lu_out,
                                           double *Kp_out) {
    double a[B], t[B];
#pragma unroll
    for (int l = 0; l < B; ++l) a[l] = (double)fabsf(v[l]);
    const double S = tree_sum<B>(a);
    const double q = __dmul_rn(S, 1.0 / (double)B);
#pragma unroll
    for (int l = 0; l < B; ++l) {
        const double d = __dsub_rn(a[l], q);
        t[l] = __dmul_rn(d, d);
    }
    *Lu_out = tree_sum<B>(t);
    *S_out = S;
    if (use_l1) {
        *Kp_out = S;
    } else {
        // a*a is exact in fp64 for fp32-valued a, so fma(a,a,c) == round(a*a + c): the same
        // bits as a separately rounded multiply and add.
        double h[B / 2];
#pragma unroll
        for (int l = 0; l < B / 2; ++l) h[l] = __fma_rn(a[2 * l], a[2 * l], __dmul_rn(a[2 * l + 1], a[2 * l + 1]));
        *Kp_out = tree_sum<B / 2>(h);
    }
}

__device__ __forceinline__ float load_v(const float *W, const float *U, long long f) {
    float w = __ldg(W + f);
    if (U) w = __fadd_rn(w, __ldg(U + f));
    return w;
}

// exact keys of block j, read from global memory (sampling and threshold-bin blocks)
template <int B>
__device__ __forceinline__ void block_keys_at(const float *W, const float *U, long long j, int use_l1,
                                              double *S, double *Lu, double *Kp) {
    float v[B];
#pragma unroll
    for (int l = 0; l < B; ++l) v[l] = load_v(W, U, j * B + l);
    block_keys<B>(v, use_l1, S, Lu, Kp);
}

// which: 0 -> prune key, 1 -> L_u
template <int B>
__device__ __forceinline__ u64 exact_key(const Params &p, long long j, int which) {
    double S, Lu, Kp;
    block_keys_at<B>(p.W, p.U, j, p.use_l1, &S, &Lu, &Kp);
    return key_bits(which ? Lu : Kp);
}

// 16 consecutive floats starting at f (f % 16 == 0); zero beyond n
__device__ __forceinline__ void load16(const float *W, const float *U, long long f, long long n, float (&v)[16]) {
    if (f + 16 <= n) {
        const float4 *src = reinterpret_cast<const float4 *>(W + f);
        float4 a0 = __ldg(src), a1 = __ldg(src + 1), a2 = __ldg(src + 2), a3 = __ldg(src + 3);
        if (U) {
            const float4 *du = reinterpret_cast<const float4 *>(U + f);
            const float4 d0 = __ldg(du), d1 = __ldg(du + 1), d2 = __ldg(du + 2), d3 = __ldg(du + 3);
            a0.x = __fadd_rn(a0.x, d0.x); a0.y = __fadd_rn(a0.y, d0.y); a0.z = __fadd_rn(a0.z, d0.z); a0.w = __fadd_rn(a0.w, d0.w);
            a1.x = __fadd_rn(a1.x, d1.x); a1.y = __fadd_rn(a1.y, d1.y); a1.z = __fadd_rn(a1.z, d1.z); a1.w = __fadd_rn(a1.w, d1.w);
            a2.x = __fadd_rn(a2.x, d2.x); a2.y = __fadd_rn(a2.y, d2.y); a2.z = __fadd_rn(a2.z, d2.z); a2.w = __fadd_rn(a2.w, d2.w);
            a3.x = __fadd_rn(a3.x, d3.x); a3.y = __fadd_rn(a3.y, d3.y); a3.z = __fadd_rn(a3.z, d3.z); a3.w = __fadd_rn(a3.w, d3.w);
        }
        v[0] = a0.x; v[1] = a0.y; v[2] = a0.z; v[3] = a0.w; v[4] = a1.x; v[5] = a1.y; v[6] = a1.z; v[7] = a1.w;
        v[8] = a2.x; v[9] = a2.y; v[10] = a2.z; v[11] = a2.w; v[12] = a3.x; v[13] = a3.y; v[14] = a3.z; v[15] = a3.w;
    } else {
#pragma unroll
        for (int l = 0; l < 16; ++l) v[l] = (f + l < n) ? load_v(W, U, f + l) : 0.f;
    }
}

// ---------------------------------------------------------------------------------------------
// sample_kernel: choose the level-0 windows
// ---------------------------------------------------------------------------------------------
// Window around the `frac` quantile of n sample keys: +-4 sigma (binomial) in rank.  Returns the
// two ranks whose keys bound the window and the rank of the quantile itself.
__device__ __forceinline__ void window_ranks(int n, double frac, int *il, int *ih, int *ipos) {
    const double pos = frac * n;
    const double margin = 4.0 * sqrt(fmax(n * frac * (1.0 - frac), 0.0)) + 4.0;
    long long a = (long long)floor(pos - margin), b = (long long)ceil(pos + margin), c = (long long)pos;
    if (a < 0) a = 0;
    if (b > n - 1) b = n - 1;
    if (c > n - 1) c = n - 1;
    *il = (int)a; *ih = (int)b; *ipos = (int)c;
}

__device__ __forceinline__ void set_window(Sel *s, u64 lo, u64 hi, int nb) {
    if (hi < lo) hi = lo;
    unsigned shift = 0;
    while (((hi - lo) >> shift) >= (u64)(nb - 2)) ++shift;
    s->lo0 = lo;
    s->hi0 = hi;
    s->shift0 = shift;
}

// rank of (key, i) among the n keys in shared memory (ties ordered by position)
__device__ __forceinline__ int rank_of(const u64 *keys, int n, u64 key, int i) {
    int r = 0;
    for (int t = 0; t < n; ++t) {
        const u64 k = keys[t];
        r += (k < key || (k == key && t < i)) ? 1 : 0;
    }
    return r;
}

template <int B>
__global__ void __launch_bounds__(NSAMP) sample_kernel(Params p, long long k_unify, long long k_prune) {
    __shared__ u64 skey[NSAMP];
    __shared__ u64 s_stat[3];                  // keys at the ranks il, ih, ipos
    __shared__ int s_kept;
    const long long mb = p.n_blocks;
    const int ns = (int)(mb < (long long)NSAMP ? mb : (long long)NSAMP);
    const int i = threadIdx.x;
    u64 kp = ~0ull, ku = ~0ull;
    if (i == 0) s_kept = 0;
    if (i < ns) {
        const long long j = (long long)(((u128)(u64)i * (u128)(u64)mb) / (u128)(u64)ns);
        double S, Lu, Kp;
        block_keys_at<B>(p.W, p.U, j, p.use_l1, &S, &Lu, &Kp);
        kp = key_bits(Kp);
        ku = key_bits(Lu);
    }
    skey[i] = kp;
    __syncthreads();
    Sel *sp = &p.work->sel[0];
    Sel *su = &p.work->sel[1];
    const long long ksel_u = k_unify - k_prune;
    int il, ih, ipos;
    window_ranks(ns, (double)k_prune / (double)mb, &il, &ih, &ipos);
    if (i < ns) {
        const int r = rank_of(skey, ns, kp, i);
        if (r == il) s_stat[0] = kp;
        if (r == ih) s_stat[1] = kp;
        if (r == ipos) s_stat[2] = kp;
    }
    __syncthreads();
    const u64 That = s_stat[2];
    if (i == 0) {
        set_window(sp, s_stat[0], s_stat[1], p.nb);
        sp->mode = (k_prune == 0) ? 1u : (k_prune == mb ? 2u : 0u);
        sp->k = (u64)k_prune;
    }
    // the sample blocks that survive the (estimated) prune threshold
    const bool kept = i < ns && (k_prune == 0 || kp > That);
    __syncthreads();
    skey[i] = kept ? ku : ~0ull;
    if (kept) atomicAdd(&s_kept, 1);
    __syncthreads();
    const int nr = s_kept > 0 ? s_kept : 1;
    const long long elig = mb - k_prune;
    window_ranks(nr, elig > 0 ? (double)ksel_u / (double)elig : 0.0, &il, &ih, &ipos);
    if (i < ns) {
        const int r = rank_of(skey, ns, kept ? ku : ~0ull, i);     // dropped samples rank last
        if (r == il) s_stat[0] = skey[i];
        if (r == ih) s_stat[1] = skey[i];
    }
    __syncthreads();
    if (i == 0) {
        set_window(su, s_stat[0], s_stat[1], p.nb);
        su->mode = (ksel_u == 0) ? 1u : (ksel_u == elig ? 2u : 0u);
        su->k = (u64)ksel_u;
    }
}

// ---------------------------------------------------------------------------------------------
// finalisation helpers, run by the last CTA of a kernel (FIN_THREADS threads)
// ---------------------------------------------------------------------------------------------
// true in exactly one CTA: the one whose threads arrive last.  Everything the other CTAs wrote
// before is visible to it afterwards.
__device__ __forceinline__ bool last_block_done(unsigned *ticket) {
    __shared__ bool s_last;
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        const unsigned t = atomicAdd(ticket, 1u);
        s_last = (t == gridDim.x - 1);
    }
    __syncthreads();
    if (s_last) __threadfence();
    return s_last;
}

// find the bin holding the r-th element; hist has nb entries
__device__ void scan_hist(const unsigned *hist, int nb, u64 r, unsigned *bin_out, u64 *r_in_bin, u64 *cnt_out,
                          unsigned *err) {
    __shared__ u64 s_part[FIN_THREADS];
    const int PER = nb / FIN_THREADS;
    u64 sum = 0;
#pragma unroll 8
    for (int i = 0; i < PER; ++i) sum += ld_vol(&hist[threadIdx.x * PER + i]);
    s_part[threadIdx.x] = sum;
    __syncthreads();
    for (int off = 1; off < FIN_THREADS; off <<= 1) {
        u64 add = 0;
        if ((int)threadIdx.x >= off) add = s_part[threadIdx.x - off];
        __syncthreads();
        s_part[threadIdx.x] += add;
        __syncthreads();
    }
    const u64 incl = s_part[threadIdx.x];
    u64 run = incl - sum;
    if (threadIdx.x == FIN_THREADS - 1 && incl < r) *err = 1;
    if (run < r && r <= incl) {                              // the bin is in this thread's range
        for (int i = 0; i < PER; ++i) {
            const u64 c = ld_vol(&hist[threadIdx.x * PER + i]);
            if (run < r && r <= run + c) {
                *bin_out = threadIdx.x * PER + i;
                *r_in_bin = r - run;
                *cnt_out = c;
            }
            run += c;
        }
    }
    __syncthreads();
}

// level 0: which bin holds the k-th element; writes the bin and its composite range
__device__ void select_bin(const Params &p, Sel *s, const unsigned *hist) {
    __shared__ unsigned s_bin, s_err;
    __shared__ u64 s_r, s_cnt;
    if (threadIdx.x == 0) { s_err = 0; s_bin = 0; s_r = 0; s_cnt = 0; }
    __syncthreads();
    scan_hist(hist, p.nb, s->k, &s_bin, &s_r, &s_cnt, &s_err);
    if (threadIdx.x == 0) {
        if (s_err) atomicOr(p.dev_status, (unsigned)MWU_DEV_SELECT);
        const unsigned B = s_bin;
        u64 klo, khi;
        if (B == 0) { klo = 0; khi = s->lo0; }
        else if (B == (unsigned)p.nb - 1u) { klo = s->hi0; khi = ~0ull >> 1; }     // keys are < 2^63
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
        __threadfence();
    }
    __syncthreads();
}

// ---------------------------------------------------------------------------------------------
// classification of a block from its bin code
// ---------------------------------------------------------------------------------------------
struct SelView {
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

template <int B>
__device__ __forceinline__ bool selected(const Params &p, const SelView &s, long long j, unsigned bin,
                                         int which) {
    if (s.mode == 1u) return false;
    if (s.mode == 2u) return true;
    if (bin < s.B) return true;
    if (bin > s.B) return false;
    const u64 key = exact_key<B>(p, j, which);
    return key < s.T_key || (key == s.T_key && (u64)j <= s.T_idx);
}

// ---------------------------------------------------------------------------------------------
// stats_kernel
// ---------------------------------------------------------------------------------------------
template <int B>
__global__ void __launch_bounds__(256) stats_kernel(Params p, double *loss_u, double *loss_p, float *u_out,
                                                    unsigned *sign_bits) {
    constexpr int NBT = 16 / B;                         // blocks per thread and step
    const Sel *sp = &p.work->sel[0];
    const Sel *su = &p.work->sel[1];
    const u64 plo = sp->lo0, phi = sp->hi0, ulo = su->lo0, uhi = su->hi0;
    const unsigned psh = sp->shift0, ush = su->shift0;
    const unsigned nb = (unsigned)p.nb;
    unsigned cnt_under = 0, cnt_over = 0;
    unsigned nonfinite = 0;
    const long long n = p.n_floats;
    const long long n_units = (n + 15) / 16;
    const long long ustride = (long long)gridDim.x * blockDim.x;
    long long unit = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    float nxt[16];
    if (unit < n_units) load16(p.W, p.U, unit * 16, n, nxt);
    for (; unit < n_units; unit += ustride) {
        float v[16];
#pragma unroll
        for (int l = 0; l < 16; ++l) v[l] = nxt[l];
        // the next unit's 64 bytes travel while this one is evaluated
        if (unit + ustride < n_units) load16(p.W, p.U, (unit + ustride) * 16, n, nxt);
        unsigned ex = 0;
#pragma unroll
        for (int l = 0; l < 16; ++l) ex = max(ex, __float_as_uint(v[l]) & 0x7fffffffu);
        nonfinite |= (ex >= 0x7f800000u) ? 1u : 0u;
        // sign plane (final): bit l of this unit's half word = (v[l] < 0)
        {
            unsigned sb = 0;
#pragma unroll
            for (int l = 0; l < 16; ++l) sb |= (v[l] < 0.f ? 1u : 0u) << l;
            unsigned short *halves = reinterpret_cast<unsigned short *>(sign_bits);
            halves[unit] = (unsigned short)sb;
            if (unit == n_units - 1 && (n_units & 1)) halves[unit + 1] = 0;
        }
        unsigned code[NBT];
        float qv[NBT];                                   // q = mean|v| of every block; emit keeps the unified ones
#pragma unroll
        for (int e = 0; e < NBT; ++e) {
            double S, Lu, Kp;
            block_keys<B>(v + e * B, p.use_l1, &S, &Lu, &Kp);
            qv[e] = __double2float_rn(__dmul_rn(S, 1.0 / (double)B));
            const long long j = unit * NBT + e;
            const unsigned bu = bin_of(key_bits(Lu), ulo, uhi, ush, nb);
            const unsigned bp = bin_of(key_bits(Kp), plo, phi, psh, nb);
            code[e] = bp | (bu << 16);
            if (j < p.n_blocks) {
                if (bp == 0) ++cnt_under;
                else if (bp == nb - 1u) ++cnt_over;
                else atomicAdd(&p.hist[bp], 1u);
                if (loss_u) loss_u[j] = Lu;
                if (loss_p) loss_p[j] = Kp;
            }
        }
        const long long j0 = unit * NBT;
        if (j0 + NBT <= p.n_blocks) {
            if (NBT == 1) { p.bins[j0] = code[0]; u_out[j0] = qv[0]; }
            else if (NBT == 2) {
                *reinterpret_cast<uint2 *>(p.bins + j0) = make_uint2(code[0], code[1 % NBT]);
                *reinterpret_cast<float2 *>(u_out + j0) = make_float2(qv[0], qv[1 % NBT]);
            } else {
#pragma unroll
                for (int e = 0; e < NBT; e += 4) {
                    *reinterpret_cast<uint4 *>(p.bins + j0 + e) =
                        make_uint4(code[e % NBT], code[(e + 1) % NBT], code[(e + 2) % NBT], code[(e + 3) % NBT]);
                    *reinterpret_cast<float4 *>(u_out + j0 + e) =
                        make_float4(qv[e % NBT], qv[(e + 1) % NBT], qv[(e + 2) % NBT], qv[(e + 3) % NBT]);
                }
            }
        } else {
#pragma unroll
            for (int e = 0; e < NBT; ++e)
                if (j0 + e < p.n_blocks) { p.bins[j0 + e] = code[e]; u_out[j0 + e] = qv[e]; }
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
    if (nonfinite) atomicOr(p.dev_status, (unsigned)MWU_DEV_NONFINITE);
    __syncthreads();
    if (threadIdx.x == 0) {
        if (s_under) atomicAdd(&p.hist[0], s_under);
        if (s_over) atomicAdd(&p.hist[nb - 1u], s_over);
    }
}

// four consecutive bin codes starting at j4 (j4 % 4 == 0); codes beyond n read as 0
__device__ __forceinline__ void load_codes4(const unsigned *bins, long long j4, long long n, unsigned (&c)[4]) {
    if (j4 + 4 <= n) {
        const uint4 v = __ldg(reinterpret_cast<const uint4 *>(bins + j4));
        c[0] = v.x; c[1] = v.y; c[2] = v.z; c[3] = v.w;
    } else {
#pragma unroll
        for (int e = 0; e < 4; ++e) c[e] = (j4 + e < n) ? __ldg(bins + j4 + e) : 0u;
    }
}

// ---------------------------------------------------------------------------------------------
// collect_kernel: exact threshold element of one selection
// ---------------------------------------------------------------------------------------------
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

template <int KIND, int B>
__global__ void __launch_bounds__(FIN_THREADS) collect_kernel(Params p) {
    Sel *s = &p.work->sel[KIND];
    if (ld_vol(&s->mode) != 0u) return;
    __shared__ u64 c_key[CAP];
    __shared__ unsigned c_idx[CAP];
    __shared__ unsigned s_bin, s_err, s_n;
    __shared__ u64 s_r, s_cnt;
    const SelView pv = view_of(&p.work->sel[0]);
    const unsigned Bsel = ld_vol(&s->B);
    const bool too_many = ld_vol(&s->cnt) > (u64)CAP;
    const long long stride = (long long)gridDim.x * blockDim.x;

    if (!too_many) {
        const u128 lo = from_halves(ld_vol(&s->lo_hi), ld_vol(&s->lo_lo));
        const u128 hi = from_halves(ld_vol(&s->hi_hi), ld_vol(&s->hi_lo));
        for (long long j0 = ((long long)blockIdx.x * blockDim.x + threadIdx.x) * 4; j0 < p.n_blocks;
             j0 += stride * 4 * PASS_LOADS) {
            unsigned codes[PASS_LOADS][4];
#pragma unroll
            for (int q = 0; q < PASS_LOADS; ++q) load_codes4(p.bins, j0 + q * stride * 4, p.n_blocks, codes[q]);
#pragma unroll
            for (int q = 0; q < PASS_LOADS; ++q) {
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const long long j = j0 + q * stride * 4 + e;
                    const unsigned code = codes[q][e];
                    const unsigned bin = KIND ? (code >> 16) : (code & 0xffffu);
                    if (j >= p.n_blocks || bin != Bsel) continue;
                    if (KIND == 1 && selected<B>(p, pv, j, code & 0xffffu, 0)) continue;
                    const u64 key = exact_key<B>(p, j, KIND);
                    const u128 c = make_c(key, (u64)j);
                    if (c >= lo && c < hi) {
                        const unsigned slot = atomicAdd(&p.work->cand_count[KIND], 1u);
                        if (slot < (unsigned)CAP) { p.cand_key[slot] = key; p.cand_idx[slot] = (unsigned)j; }
                    }
                }
            }
        }
    }
    if (!last_block_done(&p.work->ticket[KIND ? 3 : 1])) return;

    // ---- last CTA only ----
    if (too_many) {
        // massive ties: narrow the composite range pass by pass with this CTA alone
        unsigned *rhist = p.hist + (size_t)2 * p.nb;
        for (int level = 0; level < 10; ++level) {
            if (ld_vol(&s->cnt) <= (u64)CAP) break;
            for (int i = threadIdx.x; i < p.nb; i += blockDim.x) rhist[i] = 0;
            __syncthreads();
            const u128 lo = from_halves(ld_vol(&s->lo_hi), ld_vol(&s->lo_lo));
            const u128 hi = from_halves(ld_vol(&s->hi_hi), ld_vol(&s->hi_lo));
            unsigned shift = 0;
            while (((hi - lo - 1) >> shift) >= (u128)p.nb) ++shift;
            for (long long j = threadIdx.x; j < p.n_blocks; j += blockDim.x) {
                const unsigned code = ld_vol(p.bins + j);
                const unsigned bin = KIND ? (code >> 16) : (code & 0xffffu);
                if (bin != Bsel) continue;
                if (KIND == 1 && selected<B>(p, pv, j, code & 0xffffu, 0)) continue;
                const u128 c = make_c(exact_key<B>(p, j, KIND), (u64)j);
                if (c >= lo && c < hi) atomicAdd(&rhist[(unsigned)((c - lo) >> shift)], 1u);
            }
            __threadfence();
            __syncthreads();
            if (threadIdx.x == 0) s_err = 0;
            __syncthreads();
            scan_hist(rhist, p.nb, ld_vol(&s->r), &s_bin, &s_r, &s_cnt, &s_err);
            if (threadIdx.x == 0) {
                if (s_err) atomicOr(p.dev_status, (unsigned)MWU_DEV_SELECT);
                u128 nlo = lo + ((u128)s_bin << shift);
                u128 nhi = nlo + ((u128)1 << shift);
                if (nhi > hi) nhi = hi;
                s->r = s_r;
                s->cnt = s_cnt;
                s->lo_hi = (u64)(nlo >> 64); s->lo_lo = (u64)nlo;
                s->hi_hi = (u64)(nhi >> 64); s->hi_lo = (u64)nhi;
                __threadfence();
            }
            __syncthreads();
        }
        // collect inside the narrowed range
        if (threadIdx.x == 0) s_n = 0;
        __syncthreads();
        const u128 lo = from_halves(ld_vol(&s->lo_hi), ld_vol(&s->lo_lo));
        const u128 hi = from_halves(ld_vol(&s->hi_hi), ld_vol(&s->hi_lo));
        for (long long j = threadIdx.x; j < p.n_blocks; j += blockDim.x) {
            const unsigned code = ld_vol(p.bins + j);
            const unsigned bin = KIND ? (code >> 16) : (code & 0xffffu);
            if (bin != Bsel) continue;
            if (KIND == 1 && selected<B>(p, pv, j, code & 0xffffu, 0)) continue;
            const u64 key = exact_key<B>(p, j, KIND);
            const u128 c = make_c(key, (u64)j);
            if (c >= lo && c < hi) {
                const unsigned slot = atomicAdd(&s_n, 1u);
                if (slot < (unsigned)CAP) { p.cand_key[slot] = key; p.cand_idx[slot] = (unsigned)j; }
            }
        }
        __threadfence();
        __syncthreads();
        if (threadIdx.x == 0) p.work->cand_count[KIND] = s_n;
        __syncthreads();
    }
    const unsigned n = ld_vol(&p.work->cand_count[KIND]);
    const u64 r = ld_vol(&s->r);
    const unsigned m = n < (unsigned)CAP ? n : (unsigned)CAP;
    for (int i = threadIdx.x; i < CAP; i += blockDim.x) {
        c_key[i] = (i < (int)m) ? ld_vol(&p.cand_key[i]) : ~0ull;
        c_idx[i] = (i < (int)m) ? ld_vol(&p.cand_idx[i]) : ~0u;
    }
    __syncthreads();
    int np2 = 2;
    while (np2 < (int)m) np2 <<= 1;
    sort_candidates(c_key, c_idx, np2);
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

// ---------------------------------------------------------------------------------------------
// prune_select_kernel: exact prune threshold and the L_u histogram of the survivors in one pass
// ---------------------------------------------------------------------------------------------
// Every CTA first locates the prune threshold bin from the finished histogram (all write the same
// values).  The pass over the bin codes then needs no exact key outside that bin: blocks below it
// are pruned, blocks above it survive and are counted in the L_u histogram, blocks inside it become
// candidates.  The last CTA sorts the candidates, which fixes the threshold element, counts the
// L_u bins of the candidates that survive, and locates the unify threshold bin.
template <int B>
__global__ void __launch_bounds__(FIN_THREADS) prune_select_kernel(Params p) {
    Sel *sp = &p.work->sel[0];
    Sel *su = &p.work->sel[1];
    const unsigned mode_p = ld_vol(&sp->mode), mode_u = ld_vol(&su->mode);
    if (mode_p != 0u && mode_u != 0u) return;
    __shared__ u64 c_key[CAP];
    __shared__ unsigned c_idx[CAP];
    __shared__ unsigned s_bin, s_err, s_n;
    __shared__ u64 s_r, s_cnt;
    unsigned *hist_u = p.hist + p.nb;
    if (mode_p == 0u) select_bin(p, sp, p.hist);
    const unsigned Bp = ld_vol(&sp->B);
    const bool too_many = mode_p == 0u && ld_vol(&sp->cnt) > (u64)CAP;
    const u128 lo0 = from_halves(ld_vol(&sp->lo_hi), ld_vol(&sp->lo_lo));
    const u128 hi0 = from_halves(ld_vol(&sp->hi_hi), ld_vol(&sp->hi_lo));
    const long long stride = (long long)gridDim.x * blockDim.x;
    unsigned under = 0, over = 0;
    if (mode_p != 2u) {                                   // mode 2: everything is pruned, nothing survives
        // PASS_LOADS 16-byte loads are in flight per thread before their codes are looked at
        for (long long j0 = ((long long)blockIdx.x * blockDim.x + threadIdx.x) * 4; j0 < p.n_blocks;
             j0 += stride * 4 * PASS_LOADS) {
            unsigned codes[PASS_LOADS][4];
#pragma unroll
            for (int q = 0; q < PASS_LOADS; ++q) load_codes4(p.bins, j0 + q * stride * 4, p.n_blocks, codes[q]);
#pragma unroll
            for (int q = 0; q < PASS_LOADS; ++q) {
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const long long j = j0 + q * stride * 4 + e;
                    if (j >= p.n_blocks) break;
                    const unsigned bp = codes[q][e] & 0xffffu, bu = codes[q][e] >> 16;
                    if (mode_p == 0u) {
                        if (bp < Bp) continue;                // pruned
                        if (bp == Bp) {                       // decided by the last CTA
                            if (!too_many) {
                                const u64 key = exact_key<B>(p, j, 0);
                                const u128 c = make_c(key, (u64)j);
                                if (c >= lo0 && c < hi0) {
                                    const unsigned slot = atomicAdd(&p.work->cand_count[0], 1u);
                                    if (slot < (unsigned)CAP) { p.cand_key[slot] = key; p.cand_idx[slot] = (unsigned)j; }
                                }
                            }
                            continue;
                        }
                    }
                    if (mode_u != 0u) continue;
                    if (bu == 0) ++under;
                    else if (bu == (unsigned)p.nb - 1u) ++over;
                    else atomicAdd(&hist_u[bu], 1u);
                }
            }
        }
    }
    for (int m = 16; m > 0; m >>= 1) {
        under += __shfl_xor_sync(0xffffffffu, under, m);
        over += __shfl_xor_sync(0xffffffffu, over, m);
    }
    if ((threadIdx.x & 31) == 0) {
        if (under) atomicAdd(&hist_u[0], under);
        if (over) atomicAdd(&hist_u[p.nb - 1], over);
    }
    if (!last_block_done(&p.work->ticket[1])) return;

    // ---- last CTA only ----
    if (mode_p == 0u) {
        if (too_many) {
            // massive ties: narrow the composite range pass by pass with this CTA alone
            unsigned *rhist = p.hist + (size_t)2 * p.nb;
            for (int level = 0; level < 10; ++level) {
                if (ld_vol(&sp->cnt) <= (u64)CAP) break;
                for (int i = threadIdx.x; i < p.nb; i += blockDim.x) rhist[i] = 0;
                __syncthreads();
                const u128 lo = from_halves(ld_vol(&sp->lo_hi), ld_vol(&sp->lo_lo));
                const u128 hi = from_halves(ld_vol(&sp->hi_hi), ld_vol(&sp->hi_lo));
                unsigned shift = 0;
                while (((hi - lo - 1) >> shift) >= (u128)p.nb) ++shift;
                for (long long j = threadIdx.x; j < p.n_blocks; j += blockDim.x) {
                    if ((ld_vol(p.bins + j) & 0xffffu) != Bp) continue;
                    const u128 c = make_c(exact_key<B>(p, j, 0), (u64)j);
                    if (c >= lo && c < hi) atomicAdd(&rhist[(unsigned)((c - lo) >> shift)], 1u);
                }
                __threadfence();
                __syncthreads();
                if (threadIdx.x == 0) s_err = 0;
                __syncthreads();
                scan_hist(rhist, p.nb, ld_vol(&sp->r), &s_bin, &s_r, &s_cnt, &s_err);
                if (threadIdx.x == 0) {
                    if (s_err) atomicOr(p.dev_status, (unsigned)MWU_DEV_SELECT);
                    u128 nlo = lo + ((u128)s_bin << shift);
                    u128 nhi = nlo + ((u128)1 << shift);
                    if (nhi > hi) nhi = hi;
                    sp->r = s_r;
                    sp->cnt = s_cnt;
                    sp->lo_hi = (u64)(nlo >> 64); sp->lo_lo = (u64)nlo;
                    sp->hi_hi = (u64)(nhi >> 64); sp->hi_lo = (u64)nhi;
                    __threadfence();
                }
                __syncthreads();
            }
            if (threadIdx.x == 0) s_n = 0;
            __syncthreads();
            const u128 lo = from_halves(ld_vol(&sp->lo_hi), ld_vol(&sp->lo_lo));
            const u128 hi = from_halves(ld_vol(&sp->hi_hi), ld_vol(&sp->hi_lo));
            for (long long j = threadIdx.x; j < p.n_blocks; j += blockDim.x) {
                if ((ld_vol(p.bins + j) & 0xffffu) != Bp) continue;
                const u64 key = exact_key<B>(p, j, 0);
                const u128 c = make_c(key, (u64)j);
                if (c >= lo && c < hi) {
                    const unsigned slot = atomicAdd(&s_n, 1u);
                    if (slot < (unsigned)CAP) { p.cand_key[slot] = key; p.cand_idx[slot] = (unsigned)j; }
                }
            }
            __threadfence();
            __syncthreads();
            if (threadIdx.x == 0) p.work->cand_count[0] = s_n;
            __syncthreads();
        }
        const unsigned n = ld_vol(&p.work->cand_count[0]);
        const u64 r = ld_vol(&sp->r);
        const unsigned m = n < (unsigned)CAP ? n : (unsigned)CAP;
        for (int i = threadIdx.x; i < CAP; i += blockDim.x) {
            c_key[i] = (i < (int)m) ? ld_vol(&p.cand_key[i]) : ~0ull;
            c_idx[i] = (i < (int)m) ? ld_vol(&p.cand_idx[i]) : ~0u;
        }
        __syncthreads();
        int np2 = 2;
        while (np2 < (int)m) np2 <<= 1;
        sort_candidates(c_key, c_idx, np2);
        const bool bad = n > (unsigned)CAP || r == 0 || r > (u64)m;
        if (threadIdx.x == 0) {
            if (bad) {
                atomicOr(p.dev_status, (unsigned)MWU_DEV_SELECT);
                sp->T_key = 0; sp->T_idx = 0;
            } else {
                sp->T_key = c_key[r - 1];
                sp->T_idx = (u64)c_idx[r - 1];
            }
            __threadfence();
        }
        __syncthreads();
        // the blocks of the threshold bin that survive join the L_u histogram
        if (mode_u == 0u && !bad) {
            if (!too_many) {
                for (unsigned i = (unsigned)r + threadIdx.x; i < m; i += blockDim.x)
                    atomicAdd(&hist_u[ld_vol(p.bins + c_idx[i]) >> 16], 1u);
            } else {
                const SelView pv = view_of(sp);
                for (long long j = threadIdx.x; j < p.n_blocks; j += blockDim.x) {
                    const unsigned code = ld_vol(p.bins + j);
                    if ((code & 0xffffu) != Bp) continue;
                    if (!selected<B>(p, pv, j, Bp, 0)) atomicAdd(&hist_u[code >> 16], 1u);
                }
            }
        }
        __threadfence();
        __syncthreads();
    }
    if (mode_u == 0u) select_bin(p, su, hist_u);
}

// ---------------------------------------------------------------------------------------------
// emit_kernel
// ---------------------------------------------------------------------------------------------
template <int B>
__global__ void __launch_bounds__(256, 3) emit_kernel(Params p, float *Q, float *u_out,
                                                   unsigned *pruned_bitmap, unsigned *unified_bitmap,
                                                   unsigned *sign_bits) {
    constexpr int NBT = 16 / B;
    const SelView vp = view_of(&p.work->sel[0]);
    const SelView vu = view_of(&p.work->sel[1]);
    const long long n = p.n_floats;
    const int lane = threadIdx.x & 31;
    const long long n_units = (n + 15) / 16;
    const long long n_iter = (n_units + 31) / 32 * 32;      // whole warps take part in every step
    const long long n_bm_words = (p.n_blocks + 31) / 32;
    __shared__ float4 s_stage[8][128];                       // one warp step of Q per warp
    float4 *ws = s_stage[threadIdx.x >> 5];

    for (long long unit = (long long)blockIdx.x * blockDim.x + threadIdx.x; unit < n_iter;
         unit += (long long)gridDim.x * blockDim.x) {
        const long long f = unit * 16;
        const bool warp_full = (unit - lane + 32) * 16 <= n;      // all 512 floats of this warp step exist
        unsigned code[NBT];
        const long long j0 = unit * NBT;
        if (j0 + NBT <= p.n_blocks) {
            if (NBT == 1) code[0] = __ldg(p.bins + j0);
            else if (NBT == 2) { const uint2 c = __ldg(reinterpret_cast<const uint2 *>(p.bins + j0)); code[0] = c.x; code[1 % NBT] = c.y; }
            else {
#pragma unroll
                for (int e = 0; e < NBT; e += 4) {
                    const uint4 c = __ldg(reinterpret_cast<const uint4 *>(p.bins + j0 + e));
                    code[e % NBT] = c.x; code[(e + 1) % NBT] = c.y; code[(e + 2) % NBT] = c.z; code[(e + 3) % NBT] = c.w;
                }
            }
        } else {
#pragma unroll
            for (int e = 0; e < NBT; ++e) code[e] = (j0 + e < p.n_blocks) ? __ldg(p.bins + j0 + e) : 0u;
        }
        unsigned cls_p = 0, cls_u = 0;                       // bit e: block e of this thread
        constexpr unsigned ALL = (1u << NBT) - 1u;
        unsigned valid = 0;
#pragma unroll
        for (int e = 0; e < NBT; ++e) {
            const long long j = j0 + e;
            bool pr = false, un = false;
            if (j < p.n_blocks) {
                valid |= 1u << e;
                pr = selected<B>(p, vp, j, code[e] & 0xffffu, 0);
                un = !pr && selected<B>(p, vu, j, code[e] >> 16, 1);
            }
            cls_p |= (pr ? 1u : 0u) << e;
            cls_u |= (un ? 1u : 0u) << e;
        }
        // q of the unified blocks and the sign plane come from stats_kernel; W is read again
        // only where a block keeps its own values
        float uo[NBT];
#pragma unroll
        for (int e = 0; e < NBT; ++e) uo[e] = 0.f;
        if (cls_u) {
#pragma unroll
            for (int e = 0; e < NBT; ++e)
                if ((cls_u >> e) & 1u) uo[e] = u_out[j0 + e];
        }
        if (unit < n_units) {
            if (Q) {
                float v[16];
                const bool need_v = ((~cls_p & ~cls_u) & valid & ALL) != 0u;
                if (need_v) load16(p.W, p.U, f, n, v);
                else {
#pragma unroll
                    for (int l = 0; l < 16; ++l) v[l] = 0.f;
                }
                unsigned sb = 0;
                if (cls_u) sb = reinterpret_cast<const unsigned short *>(sign_bits)[unit];
                float q[16];
#pragma unroll
                for (int e = 0; e < NBT; ++e) {
                    const bool pr = (cls_p >> e) & 1u, un = (cls_u >> e) & 1u;
#pragma unroll
                    for (int l = 0; l < B; ++l) {
                        const bool neg = (sb >> (e * B + l)) & 1u;
                        q[e * B + l] = pr ? 0.f : (un ? (neg ? -uo[e] : uo[e]) : v[e * B + l]);
                    }
                }
                if (!warp_full) {
                    if (f + 16 <= n) {
                        float4 *dst = reinterpret_cast<float4 *>(Q + f);
                        dst[0] = make_float4(q[0], q[1], q[2], q[3]);
                        dst[1] = make_float4(q[4], q[5], q[6], q[7]);
                        dst[2] = make_float4(q[8], q[9], q[10], q[11]);
                        dst[3] = make_float4(q[12], q[13], q[14], q[15]);
                    } else {
#pragma unroll
                        for (int l = 0; l < 16; ++l)
                            if (f + l < n) Q[f + l] = q[l];
                    }
                } else {
#pragma unroll
                    for (int c = 0; c < 4; ++c)
                        ws[lane * 4 + (c ^ ((lane >> 1) & 3))] = make_float4(q[4 * c], q[4 * c + 1], q[4 * c + 2], q[4 * c + 3]);
                }
            }
            if (j0 + NBT <= p.n_blocks) {
                if (NBT == 1) u_out[j0] = uo[0];
                else if (NBT == 2) *reinterpret_cast<float2 *>(u_out + j0) = make_float2(uo[0], uo[1 % NBT]);
                else {
#pragma unroll
                    for (int e = 0; e < NBT; e += 4)
                        *reinterpret_cast<float4 *>(u_out + j0 + e) =
                            make_float4(uo[e % NBT], uo[(e + 1) % NBT], uo[(e + 2) % NBT], uo[(e + 3) % NBT]);
                }
            } else {
#pragma unroll
                for (int e = 0; e < NBT; ++e)
                    if (j0 + e < p.n_blocks) u_out[j0 + e] = uo[e];
            }
        }
        // Q of a whole warp step (2 KB): 16-byte stores at a 64-byte stride reach L2 as four partial
        // writes per 64 bytes, so the step goes through shared memory and leaves as four stores of
        // 512 contiguous bytes.  Thread t keeps piece c at slot c ^ ((t >> 1) & 3): no bank conflicts.
        if (Q && warp_full) {
            __syncwarp();
            float4 *dst = reinterpret_cast<float4 *>(Q + (unit - lane) * 16);
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const int t = 8 * k + (lane >> 2), c = lane & 3;
                dst[k * 32 + lane] = ws[t * 4 + (c ^ ((t >> 1) & 3))];
            }
            __syncwarp();
        }
        // class bitmaps: the warp's 32 * NBT blocks make NBT words
        {
            const long long word0 = ((unit - lane) * NBT) >> 5;
#pragma unroll
            for (int w = 0; w < NBT; ++w) {
                const int blk = w * 32 + lane;               // block of this warp step that lane reports
                const unsigned sp = __shfl_sync(0xffffffffu, cls_p, blk / NBT);
                const unsigned su = __shfl_sync(0xffffffffu, cls_u, blk / NBT);
                const unsigned wp = __ballot_sync(0xffffffffu, (sp >> (blk % NBT)) & 1u);
                const unsigned wu = __ballot_sync(0xffffffffu, (su >> (blk % NBT)) & 1u);
                if (lane == 0 && word0 + w < n_bm_words) {
                    pruned_bitmap[word0 + w] = wp;
                    unified_bitmap[word0 + w] = wu;
                }
            }
        }
    }
}

}  // namespace proj

// ---------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------
static size_t ws_off_hist() { return align_up(sizeof(proj::Work)); }
static size_t ws_off_cand_key() { return align_up(ws_off_hist() + 3 * proj::NB_MAX * sizeof(unsigned)); }
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
    sample_kernel<B><<<1, NSAMP, 0, st>>>(p, desc->k_unify, desc->k_prune);
    const long long n_units = (p.n_floats + 15) / 16;
    const long long want = (n_units + 255) / 256;
    const long long cap_blocks = (long long)sm_count * 8;
    const int grid_stream = (int)(want < cap_blocks ? (want > 0 ? want : 1) : cap_blocks);
    stats_kernel<B><<<grid_stream, 256, 0, st>>>(p, loss_u, loss_p, u, sb);

    const long long mb = p.n_blocks;
    const long long rb = (mb + 4 * FIN_THREADS - 1) / (4 * FIN_THREADS);
    const int grid_fin = (int)(rb < (long long)sm_count ? (rb > 0 ? rb : 1) : (long long)sm_count);
    const bool need_p = desc->k_prune > 0 && desc->k_prune < mb;
    const long long ksel_u = desc->k_unify - desc->k_prune;
    const bool need_u = ksel_u > 0 && ksel_u < mb - desc->k_prune;
    if (need_p || need_u) prune_select_kernel<B><<<grid_fin, FIN_THREADS, 0, st>>>(p);
    if (need_u) collect_kernel<1, B><<<grid_fin, FIN_THREADS, 0, st>>>(p);
    emit_kernel<B><<<grid_stream, 256, 0, st>>>(p, Q, u, pb, ub, sb);
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

    p.nb = p.n_blocks <= (8ll << 20) ? proj::NB_SMALL : proj::NB_MAX;
    if (cudaMemsetAsync(ws, 0, ws_off_hist() + 3 * (size_t)p.nb * sizeof(unsigned), st) != cudaSuccess)
        return MWU_ERR_CUDA;
    cudaError_t e;
    switch (desc->block) {
        case 2: e = launch_project<2>(p, desc, Q, u, pruned_bitmap, unified_bitmap, sign_bits, loss_u, loss_p, sm_count, st); break;
        case 4: e = launch_project<4>(p, desc, Q, u, pruned_bitmap, unified_bitmap, sign_bits, loss_u, loss_p, sm_count, st); break;
        case 8: e = launch_project<8>(p, desc, Q, u, pruned_bitmap, unified_bitmap, sign_bits, loss_u, loss_p, sm_count, st); break;
        default: e = launch_project<16>(p, desc, Q, u, pruned_bitmap, unified_bitmap, sign_bits, loss_u, loss_p, sm_count, st); break;
    }
    return e == cudaSuccess ? MWU_OK : MWU_ERR_CUDA;
}
