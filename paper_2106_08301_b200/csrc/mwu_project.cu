// mwu_project: Q = Unify(W + U), the Q-step of ADMM (Algorithm 1, Eq. 7) for 1-D micro-blocks.
//
// Two pipelines give the same bits (all on the caller's stream, no host synchronisation).
//
// One-pass pipeline (MWU_ALGO_ONE_PASS; the default from ONE_PASS_MIN_BLOCKS blocks on):
//   sample_kernel   one CTA sorts the keys of <= 4096 evenly spaced blocks; for each selection
//                   (prune key, L_u of the survivors) it takes the sample quantile as a provisional
//                   threshold and the sample keys 4 sigma of rank to either side as a window.
//   pass_kernel     streams W (+U) once, evaluates the fp64 keys of every block (Section 3.1) and
//                   writes every output -- Q, u, sign plane, bitmaps -- with the class the
//                   provisional thresholds give.  A block whose key lies outside the window has
//                   its final class (as long as the exact threshold lies inside, which the counts
//                   prove afterwards); the few per cent inside go to a candidate list with their
//                   bin codes and into the window histograms.
//   list_select_kernel
//                   exact prune threshold (key, block index) from the window histogram and the
//                   list; the listed survivors complete the L_u histogram.
//   list_finish_kernel
//                   exact unify threshold; rewrites the outputs of the listed blocks whose
//                   class changed.
//   If a count shows that a threshold lies outside its window (or a tie group overflows the
//   sort buffer, or the list overflows) a flag is set and the multi-pass kernels, which are
//   always enqueued behind and otherwise return at once, redo the projection.
//
// Multi-pass pipeline (MWU_ALGO_MULTI_PASS; small tensors, and the fallback):
//   sample_kernel   as above.  The window only steers efficiency; any window gives the same result.
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
constexpr int NSAMP = 4096;        // sample blocks ranked by sample_kernel
constexpr int SAMP_THREADS = 1024;
constexpr int SAMP_PER = NSAMP / SAMP_THREADS;
static_assert(SAMP_PER == 4, "sample_select ranks one level-A key with the four threads that hold 16 samples");
constexpr int STAGE_ENTRIES = 64;  // per-warp staging of candidate-list entries in pass_kernel
constexpr long long ONE_PASS_MIN_BLOCKS = 8192;    // below: launch latency decides, multi-pass has fewer launches
constexpr int PASS_LOADS = 4;      // 16-byte loads of bin codes a thread keeps in flight in the selection passes
constexpr int FIN_THREADS = 1024;   // block size of the kernels whose last CTA finalises
static_assert(NB_MAX / FIN_THREADS <= 64, "scan_hist searches one thread's bins with one warp, two per lane");

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
    // one-pass pipeline
    unsigned fcand_count[2];    // threshold-bin candidates of the two halves of resolve_kernel
    unsigned fticket[2];
    unsigned list_count;        // entries appended to the candidate list
    unsigned failed;            // != 0: the one-pass result is void, the multi-pass kernel runs
    u64 That[2];                // provisional thresholds (key bit patterns)
    unsigned release;           // resolve_kernel: the prune threshold and the unify bin are published
    unsigned bar;               // multipass_kernel: arrivals at its grid barriers (only ever grows)
    unsigned pad1[2];
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
    unsigned *hist;             // [3][nb]: prune, unify, refine scratch (multi-pass kernels)
    unsigned *fhist;            // [2][nb]: prune, unify (one-pass kernels)
    uint2 *list;                // [list_cap] candidate list: (block index, bin codes)
    unsigned list_cap;
    int gated;                  // the multi-pass kernel returns at once unless work->failed is set
    int run_sample;             // the multi-pass kernel also chooses the windows (no sample_kernel before it)
    // grouped pruning: the prune class of a block is the bit of its group (nullptr: pruning by key)
    const unsigned *gprune;     // [ceil(n_groups / 32)]
    unsigned group_rows, group_cols;     // extent of a prune group in rows and columns of W
    unsigned blocks_per_row;    // cols / b
    unsigned groups_per_row;    // cols / group_cols
    long long k_unify, k_prune;
    float *U_next;              // dual update V - Q (mwu_admm_step), else null
    double *resid;              // ||V - Q||_F^2 accumulator (mwu_admm_step), else null
    u64 *cand_key;              // [CAP]
    unsigned *cand_idx;         // [2 * CAP]
    unsigned *cand_aux;         // [2 * CAP] what resolve_kernel wants to know about a candidate besides its key
    u64 *samp_kp, *samp_ku;     // [NSAMP] each: keys of the sample blocks (one-pass pipeline)
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

// Fresh copy of the selection state in shared memory, made by the whole CTA.  Inside a kernel that
// spans several phases (grid barriers between them) plain loads of words another CTA has written
// may be served from a stale L1 line, so every phase reads its own copy, taken with volatile loads.
__device__ __forceinline__ void load_work(const Work *g, Work *s) {
    __syncthreads();
    const volatile unsigned *src = reinterpret_cast<const volatile unsigned *>(g);
    unsigned *dst = reinterpret_cast<unsigned *>(s);
    for (unsigned i = threadIdx.x; i < sizeof(Work) / 4; i += blockDim.x) dst[i] = src[i];
    __syncthreads();
}

// grouped pruning: is block j inside a pruned group?
__device__ __forceinline__ bool group_pruned(const Params &p, unsigned j) {
    const unsigned row = j / p.blocks_per_row, kb = j - row * p.blocks_per_row;
    const unsigned g = (row / p.group_rows) * p.groups_per_row + (kb * (unsigned)p.b) / p.group_cols;
    return (__ldg(p.gprune + (g >> 5)) >> (g & 31u)) & 1u;
}

// Barrier over all CTAs of a cooperative launch (all resident at once).  `counter` only grows:
// the k-th barrier of a kernel is passed when it reaches k * gridDim.x.  The wait is bounded: when
// it runs out the caller raises MWU_DEV_TIMEOUT and leaves.
constexpr long long GRID_WAIT_CYCLES = 4000000000ll;          // about two seconds
__device__ __forceinline__ bool grid_sync(unsigned *counter, unsigned k) {
    __shared__ int s_grid_ok;
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        atomicAdd(counter, 1u);
        const unsigned target = k * gridDim.x;
        int ok = 1;
        const long long t0 = clock64();
        unsigned spins = 0;
        while (ld_vol(counter) < target) {
            if ((++spins & 63u) == 0u && clock64() - t0 > GRID_WAIT_CYCLES) { ok = 0; break; }
        }
        __threadfence();
        s_grid_ok = ok;
    }
    __syncthreads();
    return s_grid_ok != 0;
}

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

// sum v^2 of a block with the same pairing as the prune key of block_keys
template <int B>
__device__ __forceinline__ double block_sumsq(const float *v) {
    double h[B / 2];
#pragma unroll
    for (int l = 0; l < B / 2; ++l) {
        const double a0 = (double)v[2 * l], a1 = (double)v[2 * l + 1];
        h[l] = __fma_rn(a0, a0, __dmul_rn(a1, a1));
    }
    return tree_sum<B / 2>(h);
}

// sum over the CTA of one double per thread, added to *dst by one thread
__device__ __forceinline__ void block_add_double(double x, double *dst) {
    __shared__ double s_part[32];
    for (int m = 16; m > 0; m >>= 1) x += __shfl_xor_sync(0xffffffffu, x, m);
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    if (lane == 0) s_part[wid] = x;
    __syncthreads();
    if (wid == 0) {
        const int nw = (blockDim.x + 31) >> 5;
        double t = lane < nw ? s_part[lane] : 0.0;
        for (int m = 16; m > 0; m >>= 1) t += __shfl_xor_sync(0xffffffffu, t, m);
        if (lane == 0 && t != 0.0) atomicAdd(dst, t);
    }
}

__device__ __forceinline__ float load_v(const float *W, const float *U, long long f) {
    float w = __ldg(W + f);
    if (U) w = __fadd_rn(w, __ldg(U + f));
    return w;
}

// the B values of block j with the widest loads its alignment allows (a block starts at a
// multiple of 4*B bytes): scalar loads of scattered blocks cost one cache-line lookup per value
template <int B>
__device__ __forceinline__ void load_block(const float *W, const float *U, long long j, float (&v)[B]) {
    if (B == 2) {
        float2 a = __ldg(reinterpret_cast<const float2 *>(W) + j);
        if (U) {
            const float2 d = __ldg(reinterpret_cast<const float2 *>(U) + j);
            a.x = __fadd_rn(a.x, d.x); a.y = __fadd_rn(a.y, d.y);
        }
        v[0] = a.x; v[1 % B] = a.y;
    } else {
#pragma unroll
        for (int c = 0; c < B / 4; ++c) {
            float4 a = __ldg(reinterpret_cast<const float4 *>(W) + j * (B / 4) + c);
            if (U) {
                const float4 d = __ldg(reinterpret_cast<const float4 *>(U) + j * (B / 4) + c);
                a.x = __fadd_rn(a.x, d.x); a.y = __fadd_rn(a.y, d.y); a.z = __fadd_rn(a.z, d.z); a.w = __fadd_rn(a.w, d.w);
            }
            v[(4 * c) % B] = a.x; v[(4 * c + 1) % B] = a.y; v[(4 * c + 2) % B] = a.z; v[(4 * c + 3) % B] = a.w;
        }
    }
}

// Approximate keys of block j in fp32, for the sample only: the sample steers the windows (any
// window gives the same result), so its keys need no more than a few good digits, and sample_kernel,
// a single CTA, has one SM's fp64 units.
template <int B>
__device__ __forceinline__ void block_keys_sample(const float *W, const float *U, long long j, int use_l1, u64 *kp,
                                                  u64 *ku) {
    float v[B];
    load_block<B>(W, U, j, v);
    float S = 0.f, sq = 0.f;
#pragma unroll
    for (int l = 0; l < B; ++l) { S += fabsf(v[l]); sq = fmaf(v[l], v[l], sq); }
    const float q = S * (1.f / (float)B);
    float lu = 0.f;
#pragma unroll
    for (int l = 0; l < B; ++l) { const float d = fabsf(v[l]) - q; lu = fmaf(d, d, lu); }
    *kp = key_bits((double)(use_l1 ? S : sq));
    *ku = key_bits((double)lu);
}

// exact keys of block j, read from global memory (threshold-bin blocks)
template <int B>
__device__ __forceinline__ void block_keys_at(const float *W, const float *U, long long j, int use_l1,
                                              double *S, double *Lu, double *Kp) {
    float v[B];
    load_block<B>(W, U, j, v);
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
__device__ __forceinline__ void set_window(Sel *s, u64 lo, u64 hi, int nb) {
    if (hi < lo) hi = lo;
    const int width = 64 - __clzll((long long)(hi - lo));
    unsigned shift = width > 16 ? (unsigned)(width - 16) : 0u;         // nb - 2 < 2^16: start just below
    while (((hi - lo) >> shift) >= (u64)(nb - 2)) ++shift;
    s->lo0 = lo;
    s->hi0 = hi;
    s->shift0 = shift;
}

// inclusive prefix sum over the CTA's SAMP_THREADS values (one per thread)
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

// Window around the `frac` quantile of n sample keys: +-4 sigma (binomial) in rank.  Returns the
// two ranks whose keys bound the window and the rank of the quantile itself.
__device__ __forceinline__ void window_ranks_f(int n, float frac, int *il, int *ih, int *ipos) {
    const float pos = frac * (float)n;
    const float margin = 4.f * sqrtf(fmaxf((float)n * frac * (1.f - frac), 0.f)) + 4.f;
    int a = (int)floorf(pos - margin), b = (int)ceilf(pos + margin), c = (int)pos;
    if (a < 0) a = 0;
    if (b > n - 1) b = n - 1;
    if (c > n - 1) c = n - 1;
    if (c < 0) c = 0;
    *il = a; *ih = b; *ipos = c;
}

// One selection of sample_kernel.  key[t] / valid[t]: this thread's sample keys; `frac` of the
// valid ones are to be selected.  Level A ranks a 1-in-16 subsample (<= 256 keys) to get a coarse
// window; level B counts all valid samples in SAMP_THREADS bins across that window and reads the
// final window [lo, hi) and the provisional threshold from the bin edges.
__device__ void sample_select(const u64 (&key)[SAMP_PER], const bool (&valid)[SAMP_PER], float frac,
                              u64 *lo_out, u64 *hi_out, u64 *t_out) {
    constexpr int NA = NSAMP / 16;
    // level-A keys, shortened to the top 24 bits below the (clear) sign bit, with the key's index in
    // the low byte: distinct words, one 32-bit compare per pair; invalid keys rank last
    __shared__ __align__(16) unsigned s_a[NA];
    __shared__ unsigned s_edge[2];                    // shortened keys at the coarse window's ranks
    __shared__ unsigned s_hist[SAMP_THREADS + 2];     // [0] under, [1 .. SAMP_THREADS] window, [+1] over
    __shared__ unsigned s_warp[32];
    __shared__ unsigned s_nvalid;
    __shared__ u64 s_res[3];
    static_assert(NA == 256, "the index of a level-A key fills the low byte of its shortened form");
    const int tid = threadIdx.x;
    if (tid == 0) s_nvalid = 0;
    for (int i = tid; i < SAMP_THREADS + 2; i += SAMP_THREADS) s_hist[i] = 0;
    // level A: sample index 16 * a is slot 0 of thread 4 * a
    const bool is_a = (tid % 4) == 0;
    const int a = tid / 4;
    const bool a_valid = is_a && valid[0];
    if (is_a) s_a[a] = a_valid ? ((unsigned)(key[0] >> 39) << 8) | (unsigned)a : 0xffffffffu;
    int nv = 0;
#pragma unroll
    for (int t = 0; t < SAMP_PER; ++t) nv += valid[t] ? 1 : 0;
    for (int m = 16; m > 0; m >>= 1) nv += __shfl_xor_sync(0xffffffffu, nv, m);
    const int na_raw = __syncthreads_count(a_valid);           // also orders the stores above
    if ((tid & 31) == 0 && nv) atomicAdd(&s_nvalid, (unsigned)nv);
    const int na = na_raw > 0 ? na_raw : 1;
    int il, ih, ipos;
    window_ranks_f(na, frac, &il, &ih, &ipos);
    {
        // four threads rank one level-A key, each against a quarter of the keys (every fourth
        // group of four: the four threads read 64 contiguous bytes, no bank conflict)
        const int part = tid % 4;
        const unsigned k = s_a[a];
        int r = 0;
        const uint4 *q = reinterpret_cast<const uint4 *>(s_a) + part;
#pragma unroll 4
        for (int t = 0; t < NA / 16; ++t) {
            const uint4 x = q[4 * t];
            r += (x.x < k ? 1 : 0) + (x.y < k ? 1 : 0) + (x.z < k ? 1 : 0) + (x.w < k ? 1 : 0);
        }
        r += __shfl_xor_sync(0xffffffffu, r, 1);
        r += __shfl_xor_sync(0xffffffffu, r, 2);
        if (is_a) {
            if (r == il) s_edge[0] = k;
            if (r == ih) s_edge[1] = k;
        }
    }
    __syncthreads();
    const int n_valid = (int)s_nvalid > 0 ? (int)s_nvalid : 1;
    // back to full keys: the low 39 bits of the edges are zero (any window is a valid window)
    u64 clo = (u64)(s_edge[0] >> 8) << 39;
    u64 chi = (u64)(s_edge[1] >> 8) << 39;
    if (s_edge[0] == 0xffffffffu) clo = ~0ull >> 1;
    if (s_edge[1] == 0xffffffffu) chi = ~0ull >> 1;
    if (chi < clo) chi = clo;
    // smallest shift with ((chi - clo) >> shift) < SAMP_THREADS (a power of two)
    const int width = 64 - __clzll((long long)(chi - clo));            // bits of chi - clo
    const unsigned shift = width > 10 ? (unsigned)(width - 10) : 0u;
    static_assert(SAMP_THREADS == 1024, "ten bits of bin index");
    // level B
    unsigned n_under = 0, n_over = 0;                 // the two catch-all counts stay in registers
#pragma unroll
    for (int t = 0; t < SAMP_PER; ++t) {
        if (!valid[t]) continue;
        const u64 k = key[t];
        if (k < clo) ++n_under;
        else if (k >= chi) ++n_over;
        else atomicAdd(&s_hist[1u + (unsigned)((k - clo) >> shift)], 1u);
    }
    for (int m = 16; m > 0; m >>= 1) {
        n_under += __shfl_xor_sync(0xffffffffu, n_under, m);
        n_over += __shfl_xor_sync(0xffffffffu, n_over, m);
    }
    if ((tid & 31) == 0) {
        if (n_under) atomicAdd(&s_hist[0], n_under);
        if (n_over) atomicAdd(&s_hist[SAMP_THREADS + 1], n_over);
    }
    __syncthreads();
    const unsigned mine = s_hist[1 + tid];
    const unsigned incl = block_scan_incl(mine, s_warp) + s_hist[0];
    const unsigned excl = incl - mine;
    window_ranks_f(n_valid, frac, &il, &ih, &ipos);
    if (tid == 0) {
        // ranks outside the coarse window keep its edge
        s_res[0] = clo;
        s_res[1] = chi;
        s_res[2] = clo;
    }
    __syncthreads();
    const u64 edge_lo = clo + ((u64)tid << shift);
    u64 edge_hi = clo + ((u64)(tid + 1) << shift);
    if (edge_hi > chi) edge_hi = chi;
    if (mine) {
        if (excl <= (unsigned)il && (unsigned)il < incl) s_res[0] = edge_lo < chi ? edge_lo : chi;
        if (excl <= (unsigned)ih && (unsigned)ih < incl) s_res[1] = edge_hi;
        if (excl <= (unsigned)ipos && (unsigned)ipos < incl) s_res[2] = edge_lo < chi ? edge_lo : chi;
    }
    __syncthreads();
    u64 lo = s_res[0], hi = s_res[1], That = s_res[2];
    if (That < lo) That = lo;
    if (hi > lo && That >= hi) That = hi - 1;         // the provisional threshold lies inside [lo, hi)
    *lo_out = lo;
    *hi_out = hi;
    *t_out = That;
    __syncthreads();
}

// block of the i-th of ns evenly spaced samples: i * mb / ns without a division (ns is either
// NSAMP, a power of two, or mb itself); i < 2^12 and mb < 2^31, so the product fits 64 bits
__device__ __forceinline__ long long sample_block(int i, long long mb, int ns) {
    static_assert((NSAMP & (NSAMP - 1)) == 0, "NSAMP is a power of two");
    return ns == NSAMP ? (long long)(((u64)i * (u64)mb) / (u64)NSAMP) : (long long)i;
}

// sample_keys_kernel: approximate keys of the NSAMP evenly spaced sample blocks, one block per
// thread, spread over many SMs (4096 scattered 64-byte reads issued by a single SM take about
// 9 us; over 32 SMs they take one memory round trip).  The same launch clears the histograms.
template <int B>
__global__ void __launch_bounds__(128) sample_keys_kernel(Params p, unsigned *zero_base, unsigned n_zero) {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const long long mb = p.n_blocks;
    const int ns = (int)(mb < (long long)NSAMP ? mb : (long long)NSAMP);
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < NSAMP) {
        u64 kp = ~0ull, ku = ~0ull;
        unsigned in_group = 0;
        if (i < ns) {
            const long long j = sample_block(i, mb, ns);
            block_keys_sample<B>(p.W, p.U, j, p.use_l1, &kp, &ku);
            if (p.gprune) in_group = group_pruned(p, (unsigned)j) ? 1u : 0u;
        }
        p.samp_kp[i] = kp;
        p.samp_ku[i] = ku | ((u64)in_group << 63);       // keys are non-negative doubles: bit 63 is free
    }
    uint4 *z = reinterpret_cast<uint4 *>(zero_base);
    for (unsigned q = blockIdx.x * blockDim.x + threadIdx.x; q < n_zero / 4; q += gridDim.x * blockDim.x)
        z[q] = make_uint4(0, 0, 0, 0);
}

// Run by one whole CTA of SAMP_THREADS threads: windows and provisional thresholds of the two
// selections, written into p.work.  from_keys: the sample keys were computed by sample_keys_kernel.
template <int B>
__device__ void sample_body(const Params &p, bool from_keys = false) {
    const long long k_unify = p.k_unify, k_prune = p.k_prune;
    const long long mb = p.n_blocks;
    const bool by_group = p.gprune != nullptr;
    const int ns = (int)(mb < (long long)NSAMP ? mb : (long long)NSAMP);
    u64 kp[SAMP_PER], ku[SAMP_PER];
    bool valid[SAMP_PER], in_group[SAMP_PER];
#pragma unroll
    for (int t = 0; t < SAMP_PER; ++t) {
        const int i = threadIdx.x * SAMP_PER + t;
        kp[t] = ~0ull;
        ku[t] = ~0ull;
        valid[t] = i < ns;
        in_group[t] = false;
        if (i < ns && from_keys) {
            kp[t] = p.samp_kp[i];
            const u64 x = p.samp_ku[i];
            ku[t] = x & (~0ull >> 1);
            in_group[t] = (x >> 63) != 0ull;
        } else if (i < ns) {
            const long long j = sample_block(i, mb, ns);
            block_keys_sample<B>(p.W, p.U, j, p.use_l1, &kp[t], &ku[t]);
            if (by_group) in_group[t] = group_pruned(p, (unsigned)j);
        }
    }
    Sel *sp = &p.work->sel[0];
    Sel *su = &p.work->sel[1];
    const long long ksel_u = k_unify - k_prune;
    u64 lo, hi, That = 0;
    if (threadIdx.x == 0 && p.resid) *p.resid = 0.0;  // the kernels that follow add to it
    if (by_group) {
        // the prune classes are known (bit of the block's group): nothing to estimate
        if (threadIdx.x == 0) {
            set_window(sp, 0, 0, p.nb);
            sp->mode = 3u;
            sp->k = (u64)k_prune;
            p.work->That[0] = 0;
        }
#pragma unroll
        for (int t = 0; t < SAMP_PER; ++t) valid[t] = valid[t] && !in_group[t];
    } else {
        sample_select(kp, valid, (float)((double)k_prune / (double)mb), &lo, &hi, &That);
        if (threadIdx.x == 0) {
            set_window(sp, lo, hi, p.nb);
            sp->mode = (k_prune == 0) ? 1u : (k_prune == mb ? 2u : 0u);
            sp->k = (u64)k_prune;
            p.work->That[0] = That;
        }
        // the sample blocks that survive the (estimated) prune threshold
#pragma unroll
        for (int t = 0; t < SAMP_PER; ++t) valid[t] = valid[t] && (k_prune == 0 || kp[t] > That);
    }
    const long long elig = mb - k_prune;
    sample_select(ku, valid, elig > 0 ? (float)((double)ksel_u / (double)elig) : 0.f, &lo, &hi, &That);
    if (threadIdx.x == 0) {
        set_window(su, lo, hi, p.nb);
        su->mode = (ksel_u == 0) ? 1u : (ksel_u == elig ? 2u : 0u);
        su->k = (u64)ksel_u;
        p.work->That[1] = That;
    }
}

// Second kernel of the one-pass pipeline (one CTA): clears the selection state and chooses the
// windows from the sample keys.  Launched with programmatic stream serialization behind
// sample_keys_kernel, and itself lets pass_kernel's CTAs start early.
template <int B>
__global__ void __launch_bounds__(SAMP_THREADS) sample_kernel(Params p) {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    unsigned *w = reinterpret_cast<unsigned *>(p.work);
    for (unsigned i = threadIdx.x; i < sizeof(Work) / 4; i += blockDim.x) w[i] = 0u;
    asm volatile("griddepcontrol.wait;" ::: "memory");     // the sample keys are complete and visible
    __syncthreads();
    sample_body<B>(p, true);
}

// ---------------------------------------------------------------------------------------------
// finalisation helpers, run by the last CTA of a kernel (FIN_THREADS threads)
// ---------------------------------------------------------------------------------------------
// true in exactly one CTA: the one whose threads arrive last.  Everything the other CTAs wrote
// before is visible to it afterwards.
__device__ __forceinline__ bool last_block_done(unsigned *ticket) {
    __shared__ bool s_last;
    __syncthreads();                       // every write of this CTA happens before thread 0's fence
    if (threadIdx.x == 0) {
        __threadfence();                   // cumulative: publishes what the barrier made visible to thread 0
        const unsigned t = atomicAdd(ticket, 1u);
        s_last = (t == gridDim.x - 1);
        if (s_last) __threadfence();
    }
    __syncthreads();
    return s_last;
}

// find the bin holding the r-th element; hist has nb entries
// `extra` (shared memory, n_extra bin numbers, may be null): one more element in each of these bins,
// counted on top of what the histogram holds (the CTA's own corrections, not yet in global memory).
__device__ void scan_hist(const unsigned *hist, int nb, u64 r, unsigned *bin_out, u64 *r_in_bin, u64 *cnt_out,
                          unsigned *err, const unsigned *extra = nullptr, unsigned n_extra = 0) {
    __shared__ u64 s_part[32];
    const int PER = nb / FIN_THREADS;
    u64 sum = 0;
    unsigned mine8[8];                                       // this thread's bins when there are eight of them
    if (PER == 8) {
        // two 16-byte loads that bypass L1 (the histogram may have been updated by other CTAs of this kernel)
        const uint4 h0 = __ldcg(reinterpret_cast<const uint4 *>(hist) + threadIdx.x * 2);
        const uint4 h1 = __ldcg(reinterpret_cast<const uint4 *>(hist) + threadIdx.x * 2 + 1);
        mine8[0] = h0.x; mine8[1] = h0.y; mine8[2] = h0.z; mine8[3] = h0.w;
        mine8[4] = h1.x; mine8[5] = h1.y; mine8[6] = h1.z; mine8[7] = h1.w;
        for (unsigned x = 0; x < n_extra; ++x) {
            const unsigned bx = extra[x];
            if ((bx >> 3) == threadIdx.x) {
#pragma unroll
                for (int i = 0; i < 8; ++i) mine8[i] += ((bx & 7u) == (unsigned)i) ? 1u : 0u;
            }
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) sum += mine8[i];
    } else if (PER == 64) {
        // A thread's 64 bins are 256 bytes: read by the thread itself, every load of a warp would
        // touch 32 cache lines (the L1 tag stage then takes 65 000 cycles per CTA for 65536 bins).
        // The warp sums them together instead: two coalesced loads and a shuffle tree per thread.
        const int l = threadIdx.x & 31, w = threadIdx.x >> 5;
#pragma unroll 4
        for (int e = 0; e < 32; ++e) {
            const int base = (w * 32 + e) * 64;
            unsigned a = ld_vol(&hist[base + l]) + ld_vol(&hist[base + 32 + l]);
            for (int m = 16; m > 0; m >>= 1) a += __shfl_xor_sync(0xffffffffu, a, m);
            if (l == e) sum = a;
        }
        for (unsigned x = 0; x < n_extra; ++x) sum += ((extra[x] >> 6) == threadIdx.x) ? 1u : 0u;
    } else {
#pragma unroll 8
        for (int i = 0; i < PER; ++i) sum += ld_vol(&hist[threadIdx.x * PER + i]);
        for (unsigned x = 0; x < n_extra; ++x) sum += (extra[x] / (unsigned)PER == threadIdx.x) ? 1u : 0u;
    }
    // inclusive scan of the per-thread sums: shuffles inside a warp, then over the 32 warp totals
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    u64 incl = sum;
    for (int m = 1; m < 32; m <<= 1) {
        const u64 y = __shfl_up_sync(0xffffffffu, incl, m);
        if (lane >= m) incl += y;
    }
    __syncthreads();                                         // s_part may still be read by an earlier call
    if (lane == 31) s_part[wid] = incl;
    __syncthreads();
    if (wid == 0) {
        u64 t = s_part[lane];
        for (int m = 1; m < 32; m <<= 1) {
            const u64 y = __shfl_up_sync(0xffffffffu, t, m);
            if (lane >= m) t += y;
        }
        s_part[lane] = t;
    }
    __syncthreads();
    if (wid) incl += s_part[wid - 1];
    const u64 run = incl - sum;
    if (threadIdx.x == FIN_THREADS - 1 && incl < r) *err = 1;
    if (PER == 8) {
        // the thread whose range holds the r-th element finds the bin among its eight counts
        if (run < r && r <= incl) {
            u64 before = run;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const u64 c = mine8[i];
                if (before < r && r <= before + c) { *bin_out = threadIdx.x * 8 + i; *r_in_bin = r - before; *cnt_out = c; }
                before += c;
            }
        }
        __syncthreads();
        return;
    }
    __shared__ int s_owner;
    __shared__ u64 s_run;
    if (threadIdx.x == 0) s_owner = -1;
    __syncthreads();
    if (run < r && r <= incl) { s_owner = threadIdx.x; s_run = run; }     // the bin is in this thread's range
    __syncthreads();
    // warp 0 scans the owner's PER (<= 64) bins together
    if (wid == 0 && s_owner >= 0) {
        const int base = s_owner * PER;
        u64 c0 = lane < PER ? (u64)ld_vol(&hist[base + lane]) : 0ull;
        u64 c1 = lane + 32 < PER ? (u64)ld_vol(&hist[base + lane + 32]) : 0ull;
        for (unsigned x = 0; x < n_extra; ++x) {
            c0 += (extra[x] == (unsigned)(base + lane)) ? 1u : 0u;
            c1 += (extra[x] == (unsigned)(base + lane + 32)) ? 1u : 0u;
        }
        u64 i0 = c0;                                   // inclusive scan over bins 0..31, then 32..63
        for (int m = 1; m < 32; m <<= 1) {
            const u64 y = __shfl_up_sync(0xffffffffu, i0, m);
            if (lane >= m) i0 += y;
        }
        const u64 tot0 = __shfl_sync(0xffffffffu, i0, 31);
        u64 i1 = c1;
        for (int m = 1; m < 32; m <<= 1) {
            const u64 y = __shfl_up_sync(0xffffffffu, i1, m);
            if (lane >= m) i1 += y;
        }
        i1 += tot0;
        const u64 before0 = s_run + i0 - c0, before1 = s_run + i1 - c1;
        if (c0 && before0 < r && r <= before0 + c0) { *bin_out = base + lane; *r_in_bin = r - before0; *cnt_out = c0; }
        if (c1 && before1 < r && r <= before1 + c1) { *bin_out = base + lane + 32; *r_in_bin = r - before1; *cnt_out = c1; }
    }
    __syncthreads();
}

// what select_bin found, kept in shared memory for the CTA that ran it
struct BinSel {
    unsigned B;
    u64 r, cnt;
    u64 lo_hi, lo_lo, hi_hi, hi_lo;
};

// level 0: which bin holds the k-th element; writes the bin and its composite range
// sr: the CTA's copy of the selection (count and window); s: the global one, written when `publish`
__device__ void select_bin(const Params &p, const Sel *sr, Sel *s, const unsigned *hist, BinSel *out, bool publish,
                           const unsigned *extra = nullptr, unsigned n_extra = 0) {
    __shared__ unsigned s_bin, s_err;
    __shared__ u64 s_r, s_cnt;
    if (threadIdx.x == 0) { s_err = 0; s_bin = 0; s_r = 0; s_cnt = 0; }
    __syncthreads();
    scan_hist(hist, p.nb, sr->k, &s_bin, &s_r, &s_cnt, &s_err, extra, n_extra);
    if (threadIdx.x == 0) {
        if (s_err) atomicOr(p.dev_status, (unsigned)MWU_DEV_SELECT);
        const unsigned B = s_bin;
        u64 klo, khi;
        if (B == 0) { klo = 0; khi = sr->lo0; }
        else if (B == (unsigned)p.nb - 1u) { klo = sr->hi0; khi = ~0ull >> 1; }     // keys are < 2^63
        else {
            klo = sr->lo0 + ((u64)(B - 1) << sr->shift0);
            khi = sr->lo0 + ((u64)B << sr->shift0);
            if (khi > sr->hi0) khi = sr->hi0;
        }
        const u128 lo = make_c(klo, 0), hi = make_c(khi, 0);
        if (publish) {                                   // for the phases that follow
            s->B = B;
            s->r = s_r;
            s->cnt = s_cnt;
            s->lo_hi = (u64)(lo >> 64); s->lo_lo = (u64)lo;
            s->hi_hi = (u64)(hi >> 64); s->hi_lo = (u64)hi;
        }
        out->B = B; out->r = s_r; out->cnt = s_cnt;
        out->lo_hi = (u64)(lo >> 64); out->lo_lo = (u64)lo;
        out->hi_hi = (u64)(hi >> 64); out->hi_lo = (u64)hi;
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

// Selection state written by an EARLIER kernel: plain (L1-cached) loads.  Volatile loads of one
// address by every warp of a large grid all queue at one L2 slice -- tens of microseconds.
__device__ __forceinline__ SelView view_of(const Sel *s) {
    SelView v;
    v.mode = s->mode;
    v.B = s->B;
    v.T_key = s->T_key;
    v.T_idx = s->T_idx;
    return v;
}

// the same, for state written earlier in the running kernel (read by one CTA only)
__device__ __forceinline__ SelView view_vol(const Sel *s) {
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
    if (s.mode == 3u) return group_pruned(p, (unsigned)j);      // grouped pruning: the group's bit
    if (bin < s.B) return true;
    if (bin > s.B) return false;
    const u64 key = exact_key<B>(p, j, which);
    return key < s.T_key || (key == s.T_key && (u64)j <= s.T_idx);
}

// ---------------------------------------------------------------------------------------------
// stats_kernel
// ---------------------------------------------------------------------------------------------
template <int B>
__device__ void stats_body(const Params &p, const Work &w, double *loss_u, double *loss_p, float *u_out,
                           unsigned *sign_bits) {
    if (p.gated && p.resid && blockIdx.x == 0 && threadIdx.x == 0) *p.resid = 0.0;   // emit_body sums afresh
    constexpr int NBT = 16 / B;                         // blocks per thread and step
    const Sel *sp = &w.sel[0];
    const Sel *su = &w.sel[1];
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
        const uint4 v = __ldcg(reinterpret_cast<const uint4 *>(bins + j4));
        c[0] = v.x; c[1] = v.y; c[2] = v.z; c[3] = v.w;
    } else {
#pragma unroll
        for (int e = 0; e < 4; ++e) c[e] = (j4 + e < n) ? __ldcg(bins + j4 + e) : 0u;
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

// Exact threshold element of selection KIND.  w: this phase's copy of the selection state;
// c_key / c_idx: CAP entries of shared memory each.
template <int KIND, int B>
__device__ void collect_body(const Params &p, const Work &w, u64 *c_key, unsigned *c_idx) {
    Sel *s = &p.work->sel[KIND];
    const Sel *sw = &w.sel[KIND];
    if (sw->mode != 0u) return;                       // the same in every CTA
    __shared__ unsigned s_bin, s_err, s_n;
    __shared__ u64 s_r, s_cnt;
    const SelView pv = view_of(&w.sel[0]);
    const unsigned Bsel = sw->B;
    const bool too_many = sw->cnt > (u64)CAP;
    const long long stride = (long long)gridDim.x * blockDim.x;

    if (!too_many) {
        const u128 lo = from_halves(sw->lo_hi, sw->lo_lo);
        const u128 hi = from_halves(sw->hi_hi, sw->hi_lo);
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
__device__ void prune_select_body(const Params &p, const Work &w, u64 *c_key, unsigned *c_idx) {
    Sel *sp = &p.work->sel[0];
    Sel *su = &p.work->sel[1];
    const unsigned mode_p = w.sel[0].mode, mode_u = w.sel[1].mode;
    if (mode_p != 0u && mode_u != 0u) return;         // the same in every CTA
    __shared__ unsigned s_bin, s_err, s_n;
    __shared__ u64 s_r, s_cnt;
    __shared__ BinSel s_sel;
    unsigned *hist_u = p.hist + p.nb;
    if (threadIdx.x == 0) { s_sel.B = 0; s_sel.r = 0; s_sel.cnt = 0; s_sel.lo_hi = s_sel.lo_lo = s_sel.hi_hi = s_sel.hi_lo = 0; }
    __syncthreads();
    if (mode_p == 0u) select_bin(p, &w.sel[0], sp, p.hist, &s_sel, true);
    const unsigned Bp = s_sel.B;
    const bool too_many = mode_p == 0u && s_sel.cnt > (u64)CAP;
    const u128 lo0 = from_halves(s_sel.lo_hi, s_sel.lo_lo);
    const u128 hi0 = from_halves(s_sel.hi_hi, s_sel.hi_lo);
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
                    } else if (mode_p == 3u) {
                        if (group_pruned(p, (unsigned)j)) continue;
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
                const SelView pv = view_vol(sp);
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
    if (mode_u == 0u) select_bin(p, &w.sel[1], su, hist_u, &s_sel, true);
}

// ---------------------------------------------------------------------------------------------
// emit_body
// ---------------------------------------------------------------------------------------------
// s_stage: 128 float4 of shared memory per warp of the CTA
template <int B>
__device__ void emit_body(const Params &p, const Work &w, float *Q, float *u_out, unsigned *pruned_bitmap,
                          unsigned *unified_bitmap, unsigned *sign_bits, float4 *s_stage) {
    constexpr int NBT = 16 / B;
    const SelView vp = view_of(&w.sel[0]);
    const SelView vu = view_of(&w.sel[1]);
    const long long n = p.n_floats;
    const int lane = threadIdx.x & 31;
    const long long n_units = (n + 15) / 16;
    const long long n_iter = (n_units + 31) / 32 * 32;      // whole warps take part in every step
    const long long n_bm_words = (p.n_blocks + 31) / 32;
    float4 *ws = s_stage + (threadIdx.x >> 5) * 128;         // one warp step of Q per warp
    double resid_acc = 0.0;

    for (long long unit = (long long)blockIdx.x * blockDim.x + threadIdx.x; unit < n_iter;
         unit += (long long)gridDim.x * blockDim.x) {
        const long long f = unit * 16;
        const bool warp_full = (unit - lane + 32) * 16 <= n;      // all 512 floats of this warp step exist
        unsigned code[NBT];
        const long long j0 = unit * NBT;
        if (j0 + NBT <= p.n_blocks) {
            if (NBT == 1) code[0] = __ldcg(p.bins + j0);
            else if (NBT == 2) { const uint2 c = __ldcg(reinterpret_cast<const uint2 *>(p.bins + j0)); code[0] = c.x; code[1 % NBT] = c.y; }
            else {
#pragma unroll
                for (int e = 0; e < NBT; e += 4) {
                    const uint4 c = __ldcg(reinterpret_cast<const uint4 *>(p.bins + j0 + e));
                    code[e % NBT] = c.x; code[(e + 1) % NBT] = c.y; code[(e + 2) % NBT] = c.z; code[(e + 3) % NBT] = c.w;
                }
            }
        } else {
#pragma unroll
            for (int e = 0; e < NBT; ++e) code[e] = (j0 + e < p.n_blocks) ? __ldcg(p.bins + j0 + e) : 0u;
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
        // only where a block keeps its own values (everywhere for the dual update: it needs v)
        float uo[NBT];
#pragma unroll
        for (int e = 0; e < NBT; ++e) uo[e] = 0.f;
        if (cls_u) {
#pragma unroll
            for (int e = 0; e < NBT; ++e)
                if ((cls_u >> e) & 1u) uo[e] = u_out[j0 + e];
        }
        if (unit < n_units) {
            if (Q || p.U_next || p.resid) {
                float v[16];
                const bool admm = p.U_next != nullptr || p.resid != nullptr;
                const bool need_v = admm || ((~cls_p & ~cls_u) & valid & ALL) != 0u;
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
                if (admm) {
                    // dual update V - Q and ||V - Q||^2 (loss of the block's class)
#pragma unroll
                    for (int e = 0; e < NBT; ++e) {
                        const bool pr = (cls_p >> e) & 1u, un = (cls_u >> e) & 1u;
                        if (p.resid && (pr || un)) {
                            double S, Lu, Kp;
                            block_keys<B>(v + e * B, 0, &S, &Lu, &Kp);
                            resid_acc += pr ? Kp : Lu;
                        }
                    }
                    if (p.U_next) {
                        if (f + 16 <= n) {
                            float4 *dst = reinterpret_cast<float4 *>(p.U_next + f);
#pragma unroll
                            for (int c = 0; c < 4; ++c)
                                dst[c] = make_float4(__fsub_rn(v[4 * c], q[4 * c]), __fsub_rn(v[4 * c + 1], q[4 * c + 1]),
                                                     __fsub_rn(v[4 * c + 2], q[4 * c + 2]), __fsub_rn(v[4 * c + 3], q[4 * c + 3]));
                        } else {
#pragma unroll
                            for (int l = 0; l < 16; ++l)
                                if (f + l < n) p.U_next[f + l] = __fsub_rn(v[l], q[l]);
                        }
                    }
                }
                if (Q) {
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
    if (p.resid) block_add_double(resid_acc, p.resid);
}

// ---------------------------------------------------------------------------------------------
// one-pass pipeline
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void one_pass_fail(const Params &p) { atomicExch(&p.work->failed, 1u); }

// pass_kernel: keys, provisional classes and every output in one sweep over W (+U).
// A block is a candidate when its final class is still open: its prune key lies inside the prune
// window, or it certainly survives pruning and its L_u lies inside the unify window.  Candidates
// are staged per warp with their two keys; when 32 have gathered, the whole warp turns them into
// bin codes, window-histogram counts and list entries (every lane busy), so the sweep itself only
// compares keys with the window edges.
// ADMM: also the dual update V - Q and ||V - Q||_F^2 (mwu_admm_step); a separate instantiation so
// that the plain projection keeps its register count.
template <int B, bool ADMM>
__global__ void __launch_bounds__(256) pass_kernel(Params p, float *Q, double *loss_u, double *loss_p,
                                                   float *u_out, unsigned *pruned_bitmap,
                                                   unsigned *unified_bitmap, unsigned *sign_bits) {
    constexpr int NBT = 16 / B;
    // Launched with programmatic stream serialization: the CTAs may start while sample_kernel still
    // runs.  The first 64 bytes of W do not depend on it and are requested at once; everything
    // sample_kernel writes (windows, cleared histograms) is read only behind the wait.
    const long long n = p.n_floats;
    const unsigned n_units = (unsigned)((n + 15) / 16);
    unsigned unit = blockIdx.x * blockDim.x + threadIdx.x;
    float nxt[16];
#pragma unroll
    for (int l = 0; l < 16; ++l) nxt[l] = 0.f;
    if (unit < n_units) load16(p.W, p.U, (long long)unit * 16, n, nxt);
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const Sel *sp = &p.work->sel[0];
    const Sel *su = &p.work->sel[1];
    const u64 plo = sp->lo0, phi = sp->hi0, ulo = su->lo0, uhi = su->hi0;
    const unsigned psh = sp->shift0, ush = su->shift0;
    const unsigned mode_p = sp->mode, mode_u = su->mode;
    const u64 Tp = p.work->That[0], Tu = p.work->That[1];
    const unsigned nb = (unsigned)p.nb, top = nb - 1u;
    unsigned *hist_p = p.fhist, *hist_u = p.fhist + p.nb;
    __shared__ float4 s_q[8][128];                       // one warp step of Q per warp
    // candidates waiting for a full 32-entry flush: block index and both keys
    __shared__ unsigned s_cidx[8][STAGE_ENTRIES];
    __shared__ u64 s_ckp[8][STAGE_ENTRIES], s_cku[8][STAGE_ENTRIES];
    const int lane = threadIdx.x & 31;
    float4 *wq = s_q[threadIdx.x >> 5];
    unsigned *cidx = s_cidx[threadIdx.x >> 5];
    u64 *ckp = s_ckp[threadIdx.x >> 5], *cku = s_cku[threadIdx.x >> 5];
    const unsigned lt_mask = (1u << lane) - 1u;
    unsigned fill = 0;                                   // warp-uniform
    unsigned under_p = 0, over_p = 0, under_u = 0, over_u = 0, nonfinite = 0;
    double resid_acc = 0.0;
    // fewer than 2^31 blocks of at least two values: units (16 values) and blocks count in 32 bits
    const unsigned n_iter = (n_units + 31u) / 32u * 32u;  // whole warps take part in every step
    const unsigned n_blocks = (unsigned)p.n_blocks;
    const unsigned n_bm_words = (n_blocks + 31u) / 32u;
    const unsigned ustride = gridDim.x * blockDim.x;

    // staged candidates [from, from + cnt) -> bin codes, window histograms, list entries (whole warp)
    auto flush = [&](unsigned from, unsigned cnt) {
        unsigned base = 0;
        if (lane == 0) base = atomicAdd(&p.work->list_count, cnt);
        base = __shfl_sync(0xffffffffu, base, 0);
        if (base + cnt > p.list_cap) {
            if (lane == 0) one_pass_fail(p);
            return;
        }
        if ((unsigned)lane < cnt) {
            const u64 kp = ckp[from + lane], ku = cku[from + lane];
            const unsigned bp = bin_of(kp, plo, phi, psh, nb), bu = bin_of(ku, ulo, uhi, ush, nb);
            if (mode_p == 0u && bp != 0u && bp != top) atomicAdd(&hist_p[bp], 1u);       // open because of the prune window
            else if (mode_u == 0u && bu != 0u && bu != top) atomicAdd(&hist_u[bu], 1u);  // a survivor inside the unify window
            p.list[base + lane] = make_uint2(cidx[from + lane], bp | (bu << 16));
        }
    };

    for (; unit < n_iter; unit += ustride) {
        float v[16];
#pragma unroll
        for (int l = 0; l < 16; ++l) v[l] = nxt[l];
        // the next unit's 64 bytes travel while this one is evaluated
        if (unit + ustride < n_units) load16(p.W, p.U, (long long)(unit + ustride) * 16, n, nxt);
        else {
#pragma unroll
            for (int l = 0; l < 16; ++l) nxt[l] = 0.f;
        }
        const bool live = unit < n_units;
        const bool warp_full = (long long)(unit - lane + 32u) * 16 <= n;      // all 512 floats of this warp step exist
        const unsigned j0 = unit * NBT;
        // Sign plane: bit l = (v[l] < 0).  Without a zero among the warp's values that is the IEEE sign
        // bit, gathered with one funnel shift per value; a zero (it may be -0.0) takes the compare.
        float vmin = fabsf(v[0]);
#pragma unroll
        for (int l = 1; l < 16; ++l) vmin = fminf(vmin, fabsf(v[l]));
        const bool has_zero = __any_sync(0xffffffffu, vmin == 0.f);
        unsigned sb = 0;
        if (!has_zero) {
#pragma unroll
            for (int l = 15; l >= 0; --l) sb = __funnelshift_l(__float_as_uint(v[l]), sb, 1);
        } else {
#pragma unroll
            for (int l = 0; l < 16; ++l) sb |= (v[l] < 0.f ? 1u : 0u) << l;
        }
        if (live) {
            unsigned short *halves = reinterpret_cast<unsigned short *>(sign_bits);
            halves[unit] = (unsigned short)sb;
            if (unit == n_units - 1 && (n_units & 1)) halves[unit + 1] = 0;
        }
        // grouped pruning: a unit's 16 values lie in one group (groups are at least 16 columns wide)
        const bool grp = mode_p == 3u && j0 < n_blocks && group_pruned(p, j0);
        unsigned cls_p = 0, cls_u = 0, cand = 0;             // bit e: block e of this thread
        u64 kpb[NBT], kub[NBT];
        float uo[NBT];
#pragma unroll
        for (int e = 0; e < NBT; ++e) {
            double S, Lu, Kp;
            block_keys<B>(v + e * B, p.use_l1, &S, &Lu, &Kp);
            const float qf = __double2float_rn(__dmul_rn(S, 1.0 / (double)B));
            // S = sum |v| is Inf or NaN exactly when some value of the block is
            nonfinite |= ((unsigned)__double2hiint(S) >= 0x7ff00000u) ? 1u : 0u;
            kpb[e] = key_bits(Kp);
            kub[e] = key_bits(Lu);
            uo[e] = 0.f;
            const unsigned j = j0 + e;
            if (j < n_blocks) {
                if (loss_u) loss_u[j] = Lu;
                if (loss_p) loss_p[j] = Kp;
                bool pr, survives, open = false;
                if (mode_p == 0u) {
                    const bool below = kpb[e] < plo, above = kpb[e] >= phi;
                    pr = kpb[e] <= Tp;
                    survives = above;
                    under_p += below ? 1u : 0u;
                    over_p += above ? 1u : 0u;
                    open = !(below || above);
                } else if (mode_p == 3u) {
                    pr = grp;                              // grouped pruning: the class is the group's bit
                    survives = !grp;
                } else {
                    pr = mode_p == 2u;
                    survives = mode_p == 1u;
                }
                const bool un = !pr && (mode_u == 2u || (mode_u == 0u && kub[e] <= Tu));
                if (survives && mode_u == 0u) {
                    const bool below = kub[e] < ulo, above = kub[e] >= uhi;
                    under_u += below ? 1u : 0u;
                    over_u += above ? 1u : 0u;
                    open = open || !(below || above);
                }
                cls_p |= (pr ? 1u : 0u) << e;
                cls_u |= (un ? 1u : 0u) << e;
                cand |= (open ? 1u : 0u) << e;
                if (un) uo[e] = qf;
                if (ADMM && p.resid) {
                    // squared distance of the block to its image: the loss of its (provisional) class
                    if (un) resid_acc += Lu;
                    else if (pr) resid_acc += p.use_l1 ? block_sumsq<B>(v + e * B) : Kp;
                }
            }
        }
        if (live) {
            if (j0 + NBT <= n_blocks) {
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
                    if (j0 + e < n_blocks) u_out[j0 + e] = uo[e];
            }
            if (Q || (ADMM && p.U_next)) {
                // q = v (kept), +-u (unified: magnitude u, sign of v), or +0
                float q[16];
#pragma unroll
                for (int e = 0; e < NBT; ++e) {
                    const bool pr = (cls_p >> e) & 1u, un = (cls_u >> e) & 1u;
                    const unsigned mag = un ? __float_as_uint(uo[e]) : 0u;
                    if (!has_zero) {
                        // no zero in the warp: the sign of v is its IEEE sign bit
                        const unsigned m1 = pr ? 0u : (un ? 0x80000000u : 0xffffffffu);
#pragma unroll
                        for (int l = 0; l < B; ++l) q[e * B + l] = __uint_as_float((__float_as_uint(v[e * B + l]) & m1) | mag);
                    } else {
                        const unsigned keep = (pr || un) ? 0u : 0xffffffffu;
                        const unsigned sgn = un ? 0x80000000u : 0u;
#pragma unroll
                        for (int l = 0; l < B; ++l) {
                            const int k = e * B + l;
                            q[k] = __uint_as_float((__float_as_uint(v[k]) & keep) | mag | ((sb << (31 - k)) & sgn));
                        }
                    }
                }
                const long long f = (long long)unit * 16;
                if (ADMM && p.U_next) {
                    // dual update: one fp32 subtraction per entry (v for a pruned block, +0 for a kept one)
                    if (f + 16 <= n) {
                        float4 *dst = reinterpret_cast<float4 *>(p.U_next + f);
#pragma unroll
                        for (int c = 0; c < 4; ++c)
                            dst[c] = make_float4(__fsub_rn(v[4 * c], q[4 * c]), __fsub_rn(v[4 * c + 1], q[4 * c + 1]),
                                                 __fsub_rn(v[4 * c + 2], q[4 * c + 2]), __fsub_rn(v[4 * c + 3], q[4 * c + 3]));
                    } else {
#pragma unroll
                        for (int l = 0; l < 16; ++l)
                            if (f + l < n) p.U_next[f + l] = __fsub_rn(v[l], q[l]);
                    }
                }
                if (!Q) {
                    // only the dual update was wanted
                } else if (!warp_full) {
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
                        wq[lane * 4 + (c ^ ((lane >> 1) & 3))] = make_float4(q[4 * c], q[4 * c + 1], q[4 * c + 2], q[4 * c + 3]);
                }
            }
        }
        // Q of a whole warp step (2 KB) leaves as four stores of 512 contiguous bytes: thread t keeps
        // piece c at slot c ^ ((t >> 1) & 3), so neither side has bank conflicts.
        if (Q && warp_full) {
            __syncwarp();
            float4 *dst = reinterpret_cast<float4 *>(Q + (long long)(unit - lane) * 16);
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const int t = 8 * k + (lane >> 2), c = lane & 3;
                dst[k * 32 + lane] = wq[t * 4 + (c ^ ((t >> 1) & 3))];
            }
            __syncwarp();
        }
        // class bitmaps: the warp's 32 * NBT blocks make NBT words
        {
            const unsigned word0 = ((unit - lane) * NBT) >> 5;
#pragma unroll
            for (int w = 0; w < NBT; ++w) {
                const int blk = w * 32 + lane;               // block of this warp step that lane reports
                const unsigned xp = __shfl_sync(0xffffffffu, cls_p, blk / NBT);
                const unsigned xu = __shfl_sync(0xffffffffu, cls_u, blk / NBT);
                const unsigned wp = __ballot_sync(0xffffffffu, (xp >> (blk % NBT)) & 1u);
                const unsigned wu = __ballot_sync(0xffffffffu, (xu >> (blk % NBT)) & 1u);
                if (lane == 0 && word0 + w < n_bm_words) {
                    pruned_bitmap[word0 + w] = wp;
                    unified_bitmap[word0 + w] = wu;
                }
            }
        }
        // candidates gather in the warp's staging buffer and leave 32 at a time
        if (__any_sync(0xffffffffu, cand != 0u)) {
#pragma unroll
            for (int e = 0; e < NBT; ++e) {
                const bool c = (cand >> e) & 1u;
                const unsigned bal = __ballot_sync(0xffffffffu, c);
                if (bal == 0u) continue;
                if (c) {
                    const unsigned pos = fill + __popc(bal & lt_mask);
                    // block index with the provisional class in its top bits (fewer than 2^30 blocks)
                    cidx[pos] = (j0 + e) | (((cls_p >> e) & 1u) << 31) | (((cls_u >> e) & 1u) << 30);
                    ckp[pos] = kpb[e];
                    cku[pos] = kub[e];
                }
                fill += __popc(bal);
                __syncwarp();
                if (fill >= 32u) {
                    fill -= 32u;
                    flush(fill, 32u);
                    __syncwarp();
                }
            }
        }
    }
    if (fill > 0u) flush(0u, fill);
    // block-level totals of the catch-all bins
    __shared__ unsigned s_tot[4];
    if (threadIdx.x < 4) s_tot[threadIdx.x] = 0;
    __syncthreads();
    for (int m = 16; m > 0; m >>= 1) {
        under_p += __shfl_xor_sync(0xffffffffu, under_p, m);
        over_p += __shfl_xor_sync(0xffffffffu, over_p, m);
        under_u += __shfl_xor_sync(0xffffffffu, under_u, m);
        over_u += __shfl_xor_sync(0xffffffffu, over_u, m);
    }
    if (lane == 0) {
        if (under_p) atomicAdd(&s_tot[0], under_p);
        if (over_p) atomicAdd(&s_tot[1], over_p);
        if (under_u) atomicAdd(&s_tot[2], under_u);
        if (over_u) atomicAdd(&s_tot[3], over_u);
    }
    if (nonfinite) atomicOr(p.dev_status, (unsigned)MWU_DEV_NONFINITE);
    __syncthreads();
    if (threadIdx.x == 0) {
        if (s_tot[0]) atomicAdd(&hist_p[0], s_tot[0]);
        if (s_tot[1]) atomicAdd(&hist_p[top], s_tot[1]);
        if (s_tot[2]) atomicAdd(&hist_u[0], s_tot[2]);
        if (s_tot[3]) atomicAdd(&hist_u[top], s_tot[3]);
    }
    if (ADMM && p.resid) block_add_double(resid_acc, p.resid);
}

constexpr unsigned IDX_MASK = 0x3fffffffu;           // list entry: block index; bit 31 / 30: provisional pruned / unified

// Block idx gets final class (pr, un) where pass_kernel had written (pr0, un0): bitmaps, u, Q (and
// the dual update) are rewritten.  Returns the change of ||V - Q||^2.
template <int B>
__device__ __forceinline__ double apply_class(const Params &p, float *Q, float *u_out, unsigned *pruned_bitmap,
                                              unsigned *unified_bitmap, unsigned idx, bool pr, bool un, bool pr0,
                                              bool un0) {
    const unsigned bit = 1u << (idx & 31u);
    unsigned *wp = pruned_bitmap + (idx >> 5), *wu = unified_bitmap + (idx >> 5);
    if (pr != pr0) { if (pr) atomicOr(wp, bit); else atomicAnd(wp, ~bit); }
    if (un != un0) { if (un) atomicOr(wu, bit); else atomicAnd(wu, ~bit); }
    const long long j = (long long)idx;
    float v[B];
    load_block<B>(p.W, p.U, j, v);
    double S, Lu, Kp;
    block_keys<B>(v, p.use_l1, &S, &Lu, &Kp);
    const float qf = __double2float_rn(__dmul_rn(S, 1.0 / (double)B));
    u_out[j] = un ? qf : 0.f;
#pragma unroll
    for (int l = 0; l < B; ++l) {
        const float q = pr ? 0.f : (un ? (v[l] < 0.f ? -qf : qf) : v[l]);
        if (Q) Q[j * B + l] = q;
        if (p.U_next) p.U_next[j * B + l] = __fsub_rn(v[l], q);
    }
    // change of ||V - Q||^2: the loss of the new class minus that of the provisional one
    if (!p.resid) return 0.0;
    const double sq = p.use_l1 ? block_sumsq<B>(v) : Kp;
    return (pr ? sq : (un ? Lu : 0.0)) - (pr0 ? sq : (un0 ? Lu : 0.0));
}

constexpr int MP_SMEM_BYTES = (FIN_THREADS / 32) * 128 * 16;     // emit staging: 2 KB per warp
constexpr int CHG_PER_THREAD = 3;                    // list entries a thread classifies before the changed ones are applied
static_assert(MP_SMEM_BYTES >= CAP * 20 + CHG_PER_THREAD * FIN_THREADS * 8,
              "candidate buffers, corrections and the compaction buffer share the staging memory");

// The multi-pass projection as a sequence of phases separated by grid barriers (cooperative launch):
// [windows from a sample] -> statistics -> prune threshold -> unify threshold -> emit.  k counts the
// barriers of the running kernel that have been passed.
template <int B>
__device__ void multipass_phases(const Params &p, Work &w, unsigned &k, bool run_sample, unsigned char *smem, float *Q,
                                 double *loss_u, double *loss_p, float *u_out, unsigned *pruned_bitmap,
                                 unsigned *unified_bitmap, unsigned *sign_bits) {
    u64 *c_key = reinterpret_cast<u64 *>(smem);
    unsigned *c_idx = reinterpret_cast<unsigned *>(smem + CAP * sizeof(u64));
    bool ok = true;
    if (run_sample) {
        if (blockIdx.x == 0) sample_body<B>(p);
        ok = grid_sync(&p.work->bar, ++k);
    }
    if (ok) {
        load_work(p.work, &w);
        stats_body<B>(p, w, loss_u, loss_p, u_out, sign_bits);
        ok = grid_sync(&p.work->bar, ++k);
    }
    if (ok) {
        prune_select_body<B>(p, w, c_key, c_idx);
        ok = grid_sync(&p.work->bar, ++k);
    }
    if (ok) {
        load_work(p.work, &w);
        collect_body<1, B>(p, w, c_key, c_idx);
        ok = grid_sync(&p.work->bar, ++k);
    }
    if (ok) {
        load_work(p.work, &w);
        emit_body<B>(p, w, Q, u_out, pruned_bitmap, unified_bitmap, sign_bits, reinterpret_cast<float4 *>(smem));
    }
    if (!ok && threadIdx.x == 0) atomicOr(p.dev_status, (unsigned)MWU_DEV_TIMEOUT);
}

// rank the m candidates in shared memory (c_key, c_idx) by (key, index); m <= CAP
// c_aux (when the candidates fit one per thread: the return value) receives g_aux in the same order
__device__ bool rank_candidates(const Params &p, const u64 *g_key, const unsigned *g_idx, const unsigned *g_aux,
                                unsigned m, u64 *c_key, unsigned *c_idx, unsigned *c_aux) {
    if (m <= blockDim.x) {
        // the usual case, a few dozen candidates: every thread ranks its own by counting
        u64 k = ~0ull;
        unsigned ix = ~0u, ax = 0u;
        if (threadIdx.x < m) {
            k = ld_vol(&g_key[threadIdx.x]);
            ix = ld_vol(&g_idx[threadIdx.x]);
            ax = ld_vol(&g_aux[threadIdx.x]);
            c_key[threadIdx.x] = k;
            c_idx[threadIdx.x] = ix;
        }
        __syncthreads();
        unsigned rank = 0;
        if (threadIdx.x < m) {
            for (unsigned t = 0; t < m; ++t) {
                const u64 x = c_key[t];
                const unsigned y = c_idx[t];
                rank += (x < k || (x == k && y < ix)) ? 1u : 0u;
            }
        }
        __syncthreads();
        if (threadIdx.x < m) { c_key[rank] = k; c_idx[rank] = ix; c_aux[rank] = ax; }
        __syncthreads();
        return true;
    }
    for (int i = threadIdx.x; i < CAP; i += blockDim.x) {
        c_key[i] = (i < (int)m) ? ld_vol(&g_key[i]) : ~0ull;
        c_idx[i] = (i < (int)m) ? ld_vol(&g_idx[i]) : ~0u;
    }
    __syncthreads();
    int np2 = 2;
    while (np2 < (int)m) np2 <<= 1;
    sort_candidates(c_key, c_idx, np2);
    return false;
}

// resolve_kernel (cooperative launch: all CTAs resident): the exact thresholds of the one-pass
// pipeline and the final classes of the listed blocks, in one launch.
//   1  every CTA finds the prune threshold bin from the window histogram (the same values in
//      all of them) and scans its slice of the list: blocks of that bin become candidates, listed
//      survivors complete the L_u histogram.
//      -- grid barrier --
//   2  every CTA ranks the few dozen candidates itself (exact threshold element, no hand-over
//      between CTAs), keeps the bins of the surviving candidates as corrections to the L_u
//      histogram, and finds the unify threshold bin.
//   3  every CTA gives the blocks of its list slice their final class: the class pass_kernel wrote
//      travels in the entry, so nothing is read for the nine in ten whose class stands; the others
//      are gathered 32 to a warp and rewritten.  Blocks of the unify threshold bin are ranked by
//      the CTA that finishes last, which fixes the threshold element and their classes.
//      -- grid barrier --
//   4  if any step gave the one-pass result up (a threshold outside its window, a threshold bin or
//      tie group too large to rank, a full list), the multi-pass phases redo the projection here.
template <int B>
__global__ void __launch_bounds__(FIN_THREADS) resolve_kernel(Params p, float *Q, double *loss_u, double *loss_p,
                                                              float *u_out, unsigned *pruned_bitmap,
                                                              unsigned *unified_bitmap, unsigned *sign_bits) {
    extern __shared__ __align__(16) unsigned char mp_smem[];
    __shared__ Work w;                                 // selection state as the earlier kernels left it
    __shared__ BinSel s_sel;
    __shared__ unsigned s_n_extra, s_n_chg;
    u64 *c_key = reinterpret_cast<u64 *>(mp_smem);
    unsigned *c_idx = reinterpret_cast<unsigned *>(mp_smem + CAP * sizeof(u64));
    unsigned *c_aux = reinterpret_cast<unsigned *>(mp_smem + CAP * 12);
    unsigned *s_extra = reinterpret_cast<unsigned *>(mp_smem + CAP * 16);               // bins of surviving candidates
    unsigned *s_chg = reinterpret_cast<unsigned *>(mp_smem + CAP * 20);                 // entries whose class changes
    unsigned k = 0;                                    // grid barriers passed
    load_work(p.work, &w);
    Sel *sp = &p.work->sel[0];
    Sel *su = &p.work->sel[1];
    const unsigned mode_p = w.sel[0].mode, mode_u = w.sel[1].mode;
    const unsigned nb = (unsigned)p.nb, top = nb - 1u;
    unsigned *hist_u = p.fhist + p.nb;
    const u64 ulo = w.sel[1].lo0, uhi = w.sel[1].hi0;
    const unsigned ush = w.sel[1].shift0;
    const unsigned n_list = min(w.list_count, p.list_cap);
    // every condition up to the second barrier is the same in all CTAs: they all take the same path
    bool alive = w.failed == 0u && !(mode_p != 0u && mode_u != 0u);
    if (threadIdx.x == 0) { s_sel.B = 0; s_sel.r = 0; s_sel.cnt = 0; s_sel.lo_hi = s_sel.lo_lo = s_sel.hi_hi = s_sel.hi_lo = 0; s_n_extra = 0; }
    __syncthreads();

    SelView vp = view_of(&w.sel[0]);
    if (alive && mode_p == 0u) {
        // ---------------- 1: the prune threshold bin, its candidates, the survivors' L_u counts ----------------
        select_bin(p, &w.sel[0], sp, p.fhist, &s_sel, blockIdx.x == 0);
        const unsigned Bp = s_sel.B;
        const u64 r_p = s_sel.r;
        // the threshold bin must be a real bin of the window and small enough to rank
        if (!(Bp >= 1u && Bp <= nb - 2u && s_sel.cnt <= (u64)CAP)) {
            if (blockIdx.x == 0 && threadIdx.x == 0) one_pass_fail(p);
            alive = false;
        }
        if (alive) {
            unsigned under = 0, over = 0;
            const u128 lo0 = from_halves(s_sel.lo_hi, s_sel.lo_lo);
            const u128 hi0 = from_halves(s_sel.hi_hi, s_sel.hi_lo);
            // a thread's entries are requested together (each iteration would otherwise wait for its own load)
            const unsigned gstride = gridDim.x * blockDim.x;
            for (unsigned i0 = blockIdx.x * blockDim.x + threadIdx.x; i0 < n_list; i0 += 4u * gstride) {
              uint2 ent[4];
#pragma unroll
              for (int t4 = 0; t4 < 4; ++t4) {
                  const unsigned i = i0 + (unsigned)t4 * gstride;
                  ent[t4] = i < n_list ? __ldg(&p.list[i]) : make_uint2(0u, 0u);      // code 0: skipped below
              }
#pragma unroll
              for (int t4 = 0; t4 < 4; ++t4) {
                const uint2 e = ent[t4];
                const unsigned idx = e.x & IDX_MASK;
                const unsigned bp = e.y & 0xffffu, bu = e.y >> 16;
                if (bp == 0u || bp == top) continue;          // not in the prune window: counted by pass_kernel
                if (bp < Bp) continue;                        // pruned
                if (bp == Bp) {                               // ranked after the barrier
                    double S, Lu, Kp;
                    block_keys_at<B>(p.W, p.U, (long long)idx, p.use_l1, &S, &Lu, &Kp);
                    const u64 key = key_bits(Kp);
                    const u128 c = make_c(key, (u64)idx);
                    if (c >= lo0 && c < hi0) {
                        const unsigned slot = atomicAdd(&p.work->fcand_count[0], 1u);
                        if (slot < (unsigned)CAP) {
                            p.cand_key[slot] = key;
                            p.cand_idx[slot] = idx;
                            p.cand_aux[slot] = bin_of(key_bits(Lu), ulo, uhi, ush, nb);   // where it counts if it survives
                        }
                    }
                    continue;
                }
                if (mode_u != 0u) continue;
                if (bu == 0u) ++under;
                else if (bu == top) ++over;
                else atomicAdd(&hist_u[bu], 1u);
              }
            }
            for (int m = 16; m > 0; m >>= 1) {
                under += __shfl_xor_sync(0xffffffffu, under, m);
                over += __shfl_xor_sync(0xffffffffu, over, m);
            }
            if ((threadIdx.x & 31) == 0) {
                if (under) atomicAdd(&hist_u[0], under);
                if (over) atomicAdd(&hist_u[top], over);
            }
        }
        if (!grid_sync(&p.work->bar, ++k)) {              // bounded; every CTA runs into the same limit
            if (threadIdx.x == 0) atomicOr(p.dev_status, (unsigned)MWU_DEV_TIMEOUT);
            return;
        }
        if (alive) {
            // ---------------- 2: exact prune threshold, corrections, unify threshold bin ----------------
            const unsigned m = ld_vol(&p.work->fcand_count[0]);
            if (m > (unsigned)CAP || r_p < 1 || r_p > (u64)m) {
                if (blockIdx.x == 0 && threadIdx.x == 0) one_pass_fail(p);
                alive = false;
            } else {
                const bool have_aux = rank_candidates(p, p.cand_key, p.cand_idx, p.cand_aux, m, c_key, c_idx, c_aux);
                vp.B = Bp;
                vp.T_key = c_key[r_p - 1];
                vp.T_idx = (u64)c_idx[r_p - 1];
                if (blockIdx.x == 0 && threadIdx.x == 0) { sp->T_key = vp.T_key; sp->T_idx = vp.T_idx; }
                // the candidates that survive belong in the L_u histogram: kept here as corrections
                if (mode_u == 0u) {
                    for (unsigned i = (unsigned)r_p + threadIdx.x; i < m; i += blockDim.x) {
                        const unsigned bu = have_aux ? c_aux[i] : bin_of(exact_key<B>(p, (long long)c_idx[i], 1), ulo, uhi, ush, nb);
                        s_extra[atomicAdd(&s_n_extra, 1u)] = bu;
                    }
                }
                __syncthreads();
            }
        }
    }
    unsigned Bu = 0;
    u64 r_u = 0;
    u128 lo = 0, hi = 0;
    if (alive && mode_u == 0u) {
        select_bin(p, &w.sel[1], su, hist_u, &s_sel, blockIdx.x == 0, s_extra, s_n_extra);
        Bu = s_sel.B;
        r_u = s_sel.r;
        lo = from_halves(s_sel.lo_hi, s_sel.lo_lo);
        hi = from_halves(s_sel.hi_hi, s_sel.hi_lo);
        if (!(Bu >= 1u && Bu <= nb - 2u && s_sel.cnt <= (u64)CAP)) {
            if (blockIdx.x == 0 && threadIdx.x == 0) one_pass_fail(p);
            alive = false;
        }
    }
    if (alive) {
        // ---------------- 3: final classes of the listed blocks ----------------
        double resid_delta = 0.0;
        const unsigned per_round = CHG_PER_THREAD * gridDim.x * blockDim.x;
        const unsigned rounds = (n_list + per_round - 1u) / per_round;
        for (unsigned rd = 0; rd < rounds; ++rd) {
            if (threadIdx.x == 0) s_n_chg = 0;
            __syncthreads();
            uint2 ent[CHG_PER_THREAD];
            bool have[CHG_PER_THREAD];
#pragma unroll
            for (int t3 = 0; t3 < CHG_PER_THREAD; ++t3) {
                const unsigned i = ((rd * CHG_PER_THREAD + t3) * gridDim.x + blockIdx.x) * blockDim.x + threadIdx.x;
                have[t3] = i < n_list;
                ent[t3] = have[t3] ? __ldg(&p.list[i]) : make_uint2(0u, 0u);
            }
#pragma unroll
            for (int t3 = 0; t3 < CHG_PER_THREAD; ++t3) {
                if (!have[t3]) continue;
                const uint2 e = ent[t3];
                const unsigned idx = e.x & IDX_MASK;
                const bool pr0 = (e.x >> 31) & 1u, un0 = (e.x >> 30) & 1u;
                const unsigned bu = e.y >> 16;
                const bool pr = selected<B>(p, vp, (long long)idx, e.y & 0xffffu, 0);
                bool un = false, held = false;
                if (!pr) {
                    if (mode_u == 2u) un = true;
                    else if (mode_u == 0u) {
                        if (bu == Bu) {                            // ranked by the last CTA
                            const u64 key = exact_key<B>(p, (long long)idx, 1);
                            const u128 c = make_c(key, (u64)idx);
                            if (c >= lo && c < hi) {
                                const unsigned slot = atomicAdd(&p.work->fcand_count[1], 1u);
                                if (slot < (unsigned)CAP) {
                                    p.cand_key[CAP + slot] = key;
                                    p.cand_idx[CAP + slot] = idx;
                                    p.cand_aux[CAP + slot] = (pr0 ? 2u : 0u) | (un0 ? 1u : 0u);   // the class pass_kernel wrote
                                }
                                held = true;
                            }
                            un = c < lo;
                        } else un = bu < Bu;
                    }
                }
                if (!held && (pr != pr0 || un != un0)) {
                    // index with the final class in bits 31 / 30, the provisional class in a second word
                    const unsigned slot = atomicAdd(&s_n_chg, 1u);
                    s_chg[2 * slot] = idx | ((pr ? 1u : 0u) << 31) | ((un ? 1u : 0u) << 30);
                    s_chg[2 * slot + 1] = (pr0 ? 2u : 0u) | (un0 ? 1u : 0u);
                }
            }
            __syncthreads();
            // the changed blocks of this round, one per thread (every lane of the leading warps busy)
            const unsigned n_chg = s_n_chg;
            for (unsigned c = threadIdx.x; c < n_chg; c += blockDim.x) {
                const unsigned pe = s_chg[2 * c], old = s_chg[2 * c + 1];
                resid_delta += apply_class<B>(p, Q, u_out, pruned_bitmap, unified_bitmap, pe & IDX_MASK, (pe >> 31) & 1u,
                                              (pe >> 30) & 1u, (old >> 1) & 1u, old & 1u);
            }
            __syncthreads();
        }
        if (p.resid) block_add_double(resid_delta, p.resid);
        if (mode_u == 0u && last_block_done(&p.work->fticket[1])) {
            // ---- the CTA that finishes last: the blocks of the unify threshold bin ----
            const unsigned m = ld_vol(&p.work->fcand_count[1]);
            if (m > (unsigned)CAP || r_u < 1 || r_u > (u64)m) {
                if (threadIdx.x == 0) one_pass_fail(p);
            } else {
                const bool have_aux = rank_candidates(p, p.cand_key + CAP, p.cand_idx + CAP, p.cand_aux + CAP, m, c_key,
                                                      c_idx, c_aux);
                if (threadIdx.x == 0) { su->T_key = c_key[r_u - 1]; su->T_idx = (u64)c_idx[r_u - 1]; }
                const unsigned r = (unsigned)r_u;
                double tail_delta = 0.0;
                for (unsigned i = threadIdx.x; i < m; i += blockDim.x) {
                    // the class pass_kernel wrote for this block: carried with the candidate, else read back
                    const unsigned idx = c_idx[i], bit = 1u << (idx & 31u);
                    const bool pr0 = have_aux ? ((c_aux[i] >> 1) & 1u) != 0u : (ld_vol(pruned_bitmap + (idx >> 5)) & bit) != 0u;
                    const bool un0 = have_aux ? (c_aux[i] & 1u) != 0u : (ld_vol(unified_bitmap + (idx >> 5)) & bit) != 0u;
                    const bool un = i < r;
                    if (pr0 || un != un0)
                        tail_delta += apply_class<B>(p, Q, u_out, pruned_bitmap, unified_bitmap, idx, false, un, pr0, un0);
                }
                if (p.resid) block_add_double(tail_delta, p.resid);
            }
        }
    }
    // ---------------- 4: the fallback, if the one-pass result was given up anywhere ----------------
    if (!grid_sync(&p.work->bar, ++k)) {
        if (threadIdx.x == 0) atomicOr(p.dev_status, (unsigned)MWU_DEV_TIMEOUT);
        return;
    }
    load_work(p.work, &w);
    if (w.failed == 0u) return;
    multipass_phases<B>(p, w, k, false, mp_smem, Q, loss_u, loss_p, u_out, pruned_bitmap, unified_bitmap, sign_bits);
}

// ---------------------------------------------------------------------------------------------
// multipass_kernel (cooperative launch): the whole multi-pass projection in one launch.  It is the
// projection of small tensors (launch latency decides there) and of MWU_ALGO_MULTI_PASS.
// ---------------------------------------------------------------------------------------------
template <int B>
__global__ void __launch_bounds__(FIN_THREADS) multipass_kernel(Params p, float *Q, double *loss_u, double *loss_p,
                                                                float *u_out, unsigned *pruned_bitmap,
                                                                unsigned *unified_bitmap, unsigned *sign_bits) {
    extern __shared__ __align__(16) unsigned char mp_smem[];
    __shared__ Work w;
    unsigned k = 0;
    multipass_phases<B>(p, w, k, p.run_sample != 0, mp_smem, Q, loss_u, loss_p, u_out, pruned_bitmap, unified_bitmap,
                        sign_bits);
}

// ---------------------------------------------------------------------------------------------
// grouped pruning: keys of the prune groups, and the groups to zero
// ---------------------------------------------------------------------------------------------
// One CTA takes 256 rows x 64 columns of W (+U).  A half warp reads 64 consecutive values of one row;
// every lane squares (or takes the magnitude of) its four values and the sums climb the pairwise tree
// over the group's columns with shuffles (the pairing of the block keys continued across blocks);
// the rows of a group are then summed as a pairwise tree in shared memory.  Everything is fp64 with
// one rounding per operation, in a fixed order: the keys do not depend on the launch shape.
template <int GC>                                      // columns of a group: 16, 32 or 64
__global__ void __launch_bounds__(256) group_stats_kernel(Params p, double *gkey, long long rows, long long cols) {
    __shared__ double s_row[256][4];
    constexpr unsigned gc = GC;
    const unsigned gr = p.group_rows;
    constexpr unsigned nsl = 64u / gc;                  // group slices per CTA tile: 4, 2 or 1
    constexpr unsigned lanes_per_slice = gc / 4u;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long row0 = (long long)blockIdx.y * 256, col0 = (long long)blockIdx.x * 64;
    const long long col = col0 + (lane & 15) * 4;
    const long long first = (row0 + warp * 32 + (lane >> 4)) * cols + col;      // this thread's rows: every second one from here
    const bool l1 = p.use_l1 != 0;
#pragma unroll 4
    for (int it = 0; it < 16; ++it) {
        const int r = warp * 32 + it * 2 + (lane >> 4);
        const long long row = row0 + r;
        const long long at = first + (long long)it * 2 * cols;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (row < rows && col < cols) {
            v = __ldg(reinterpret_cast<const float4 *>(p.W + at));
            if (p.U) {
                const float4 d = __ldg(reinterpret_cast<const float4 *>(p.U + at));
                v.x = __fadd_rn(v.x, d.x); v.y = __fadd_rn(v.y, d.y); v.z = __fadd_rn(v.z, d.z); v.w = __fadd_rn(v.w, d.w);
            }
        }
        const double a0 = (double)fabsf(v.x), a1 = (double)fabsf(v.y), a2 = (double)fabsf(v.z), a3 = (double)fabsf(v.w);
        double t;
        if (l1) t = __dadd_rn(__dadd_rn(a0, a1), __dadd_rn(a2, a3));
        else t = __dadd_rn(__fma_rn(a0, a0, __dmul_rn(a1, a1)), __fma_rn(a2, a2, __dmul_rn(a3, a3)));   // squares are exact
#pragma unroll
        for (unsigned m = 1; m < lanes_per_slice; m <<= 1) t = __dadd_rn(t, __shfl_xor_sync(0xffffffffu, t, m));
        if (((unsigned)lane & (lanes_per_slice - 1u)) == 0u) s_row[r][((unsigned)lane & 15u) / lanes_per_slice] = t;
    }
    __syncthreads();
    // rows of a group: r with r ^ 1, then r ^ 2, ...
    for (unsigned sdist = 1; sdist < gr; sdist <<= 1) {
        for (unsigned i = threadIdx.x; i < 256u * nsl; i += blockDim.x) {
            const unsigned r = i / nsl, sl = i % nsl;
            if ((r & (2u * sdist - 1u)) == 0u) s_row[r][sl] = __dadd_rn(s_row[r][sl], s_row[r + sdist][sl]);
        }
        __syncthreads();
    }
    const long long gpr = cols / gc;                    // groups per row tile
    for (unsigned i = threadIdx.x; i < (256u / gr) * nsl; i += blockDim.x) {
        const unsigned g = i / nsl, sl = i % nsl;
        const long long row = row0 + (long long)g * gr, c = col0 + (long long)sl * gc;
        if (row < rows && c < cols) gkey[(row / gr) * gpr + c / gc] = s_row[g * gr][sl];
    }
}

// One CTA: the kg groups with the smallest (key, index) get their bit in gprune.  Radix selection on
// the keys' bit patterns (eight passes of eight bits) gives the threshold key and how many groups
// holding exactly that key are taken; those are the ones with the lowest indices.
__global__ void __launch_bounds__(FIN_THREADS) group_select_kernel(const double *gkey, unsigned n_groups, unsigned kg,
                                                                   unsigned *gprune) {
    __shared__ unsigned s_hist[256];
    __shared__ u64 s_prefix;
    __shared__ unsigned s_r;
    __shared__ unsigned s_warp[32];
    const u64 *keys = reinterpret_cast<const u64 *>(gkey);
    const unsigned n_words = (n_groups + 31u) / 32u;
    if (kg == 0u || kg >= n_groups) {
        for (unsigned i = threadIdx.x; i < n_words; i += blockDim.x) {
            unsigned wv = kg == 0u ? 0u : 0xffffffffu;
            if (kg != 0u && i == n_words - 1u && (n_groups & 31u)) wv = (1u << (n_groups & 31u)) - 1u;
            gprune[i] = wv;
        }
        return;
    }
    if (threadIdx.x == 0) { s_prefix = 0; s_r = kg; }
    u64 mask = 0;
    for (int shift = 56; shift >= 0; shift -= 8) {
        for (unsigned i = threadIdx.x; i < 256u; i += blockDim.x) s_hist[i] = 0;
        __syncthreads();
        const u64 prefix = s_prefix;
        for (unsigned i = threadIdx.x; i < n_groups; i += blockDim.x) {
            const u64 k = __ldg(keys + i);
            if ((k & mask) == prefix) atomicAdd(&s_hist[(unsigned)(k >> shift) & 255u], 1u);
        }
        __syncthreads();
        if (threadIdx.x < 32) {
            // the digit holding the r-th key: eight bins a lane, a shuffle scan over the lanes
            const unsigned lane = threadIdx.x;
            unsigned mine[8], sum = 0;
#pragma unroll
            for (int j = 0; j < 8; ++j) { mine[j] = s_hist[lane * 8 + j]; sum += mine[j]; }
            unsigned incl = sum;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const unsigned t = __shfl_up_sync(0xffffffffu, incl, off);
                if (lane >= (unsigned)off) incl += t;
            }
            const unsigned r = s_r;
            const unsigned hit = __ballot_sync(0xffffffffu, incl >= r);      // never empty: the keys left are >= r
            const unsigned owner = hit ? (unsigned)__ffs(hit) - 1u : 31u;
            if (lane == owner) {
                unsigned left = r - (incl - sum), d = 0;
                while (d < 7u && mine[d] < left) { left -= mine[d]; ++d; }
                s_r = left;
                s_prefix = prefix | ((u64)(lane * 8u + d) << shift);
            }
        }
        mask |= (u64)255 << shift;
        __syncthreads();
    }
    const u64 T = s_prefix;
    const unsigned r_ties = s_r;                        // groups with key == T that are taken (>= 1)
    // every thread owns a run of whole bitmap words; ties are numbered in index order
    const unsigned words_per = (n_words + blockDim.x - 1u) / blockDim.x;
    const unsigned w0 = threadIdx.x * words_per, w1 = min(w0 + words_per, n_words);
    unsigned ties = 0;
    for (unsigned wi = w0; wi < w1; ++wi)
        for (unsigned bit = 0; bit < 32u; ++bit) {
            const unsigned i = wi * 32u + bit;
            if (i < n_groups && __ldg(keys + i) == T) ++ties;
        }
    const unsigned incl = block_scan_incl(ties, s_warp);
    unsigned ordinal = incl - ties;                     // ties before this thread's run
    for (unsigned wi = w0; wi < w1; ++wi) {
        unsigned wv = 0;
        for (unsigned bit = 0; bit < 32u; ++bit) {
            const unsigned i = wi * 32u + bit;
            if (i >= n_groups) break;
            const u64 k = __ldg(keys + i);
            bool take = k < T;
            if (k == T) { take = ordinal < r_ties; ++ordinal; }
            wv |= (take ? 1u : 0u) << bit;
        }
        gprune[wi] = wv;
    }
}

}  // namespace proj

// ---------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------
static size_t ws_off_hist() { return align_up(sizeof(proj::Work)); }
static size_t ws_off_cand_key() { return align_up(ws_off_hist() + 5 * proj::NB_MAX * sizeof(unsigned)); }
// two sets of candidates: the two halves of resolve_kernel each keep their own
static size_t ws_off_cand_idx() { return align_up(ws_off_cand_key() + 2 * proj::CAP * sizeof(proj::u64)); }
static size_t ws_off_cand_aux() { return align_up(ws_off_cand_idx() + 2 * proj::CAP * sizeof(unsigned)); }
static size_t ws_off_samp() { return align_up(ws_off_cand_aux() + 2 * proj::CAP * sizeof(unsigned)); }
static size_t ws_off_bins() { return align_up(ws_off_samp() + 2 * proj::NSAMP * sizeof(proj::u64)); }
static size_t ws_off_list(size_t mb) { return align_up(ws_off_bins() + (mb + 8) * sizeof(unsigned)); }
// candidate list of the one-pass pipeline: a quarter of the blocks (the windows hold a few per cent)
static size_t list_capacity(size_t mb) { return mb / 4 + 4096; }
static size_t ws_off_gkey(size_t mb) { return align_up(ws_off_list(mb) + list_capacity(mb) * sizeof(uint2)); }
static size_t n_groups_of(const mwu_proj_desc *d) {
    return grouped(d) ? (size_t)(d->rows / d->prune_group_rows) * (size_t)(d->cols / d->prune_group_cols) : 0;
}
static size_t ws_off_gprune(const mwu_proj_desc *d, size_t mb) { return align_up(ws_off_gkey(mb) + n_groups_of(d) * sizeof(double)); }

static bool use_one_pass(const mwu_proj_desc *desc) {
    const long long mb = desc->rows * desc->cols / desc->block;
    if (mb >= (1ll << 30)) return false;               // list entries keep two class bits above the block index
    if (desc->algo == MWU_ALGO_ONE_PASS) return true;
    if (desc->algo == MWU_ALGO_MULTI_PASS) return false;
    return mb >= proj::ONE_PASS_MIN_BLOCKS;
}

}  // namespace mwu

extern "C" size_t mwu_project_workspace_bytes(const mwu_proj_desc *desc) {
    if (mwu::validate_desc(desc, false) != MWU_OK) return 0;
    if (mwu::shape_of(desc).shaped) return mwu::shapes::workspace_bytes(desc);
    const size_t mb = (size_t)(desc->rows * desc->cols / desc->block);
    return mwu::align_up(mwu::ws_off_gprune(desc, mb) + (mwu::n_groups_of(desc) + 31) / 32 * 4 + 16);
}

// Cooperative launch (every CTA resident at once, which the grid barriers of the kernel rely on):
// the grid is cut to what the device can hold of this kernel.
template <typename... Args>
static cudaError_t launch_cooperative(void (*kern)(Args...), int grid, int threads, size_t smem, int sm_count,
                                      cudaStream_t st, Args... args) {
    int per_sm = 0;
    cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, threads, smem);
    if (e != cudaSuccess) return e;
    if (per_sm < 1) return cudaErrorCooperativeLaunchTooLarge;
    const long long cap = (long long)per_sm * sm_count;
    if (grid > cap) grid = (int)cap;
    void *argv[] = {(void *)&args...};
    mwu::count_launch();
    return cudaLaunchCooperativeKernel((const void *)kern, dim3((unsigned)grid), dim3((unsigned)threads), argv, smem, st);
}

template <int B>
static cudaError_t launch_project(const mwu::proj::Params &p, const mwu_proj_desc *desc, float *Q,
                                  float *u, unsigned *pb, unsigned *ub, unsigned *sb, double *loss_u,
                                  double *loss_p, int sm_count, bool one_pass, double *gkey, unsigned *gprune,
                                  cudaStream_t st) {
    using namespace mwu::proj;
    cudaError_t e;
    if (p.gprune) {
        // grouped pruning: the groups' keys, then the groups to zero (a bit per group)
        const dim3 grid((unsigned)((desc->cols + 63) / 64), (unsigned)((desc->rows + 255) / 256));
        switch (desc->prune_group_cols) {
            case 16: group_stats_kernel<16><<<grid, 256, 0, st>>>(p, gkey, desc->rows, desc->cols); break;
            case 32: group_stats_kernel<32><<<grid, 256, 0, st>>>(p, gkey, desc->rows, desc->cols); break;
            default: group_stats_kernel<64><<<grid, 256, 0, st>>>(p, gkey, desc->rows, desc->cols); break;
        }
        const unsigned n_groups = (unsigned)mwu::n_groups_of(desc);
        const unsigned per_group = (unsigned)(desc->prune_group_rows * desc->prune_group_cols / desc->block);
        group_select_kernel<<<1, FIN_THREADS, 0, st>>>(gkey, n_groups, (unsigned)(desc->k_prune / per_group), gprune);
        mwu::count_launch(2);
    }
    const long long n_units = (p.n_floats + 15) / 16;
    const long long want = (n_units + 255) / 256;
    const long long cap_blocks = (long long)sm_count * 8;
    const int grid_stream = (int)(want < cap_blocks ? (want > 0 ? want : 1) : cap_blocks);
    const long long mb = p.n_blocks;
    const bool need_p = !p.gprune && desc->k_prune > 0 && desc->k_prune < mb;
    const long long ksel_u = desc->k_unify - desc->k_prune;
    const bool need_u = ksel_u > 0 && ksel_u < mb - desc->k_prune;
    const long long want_mp = (n_units + FIN_THREADS - 1) / FIN_THREADS;
    const int grid_mp = (int)(want_mp < (long long)sm_count ? (want_mp > 0 ? want_mp : 1) : (long long)sm_count);
    static bool smem_set = false;                       // per instantiation: the attribute sticks to the function
    if (!smem_set) {
        e = cudaFuncSetAttribute(multipass_kernel<B>, cudaFuncAttributeMaxDynamicSharedMemorySize, MP_SMEM_BYTES);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(resolve_kernel<B>, cudaFuncAttributeMaxDynamicSharedMemorySize, MP_SMEM_BYTES);
        if (e != cudaSuccess) return e;
        smem_set = true;
    }

    if (one_pass) {
        // the sample keys (and the cleared histograms) from 32 SMs, then one CTA ranks the sample; the two
        // kernels behind are launched with programmatic stream serialization, so their CTAs are in place
        // (and the sweep's first loads in flight) when their predecessor ends
        const unsigned n_zero = 5u * (unsigned)p.nb;
        sample_keys_kernel<B><<<NSAMP / 128, 128, 0, st>>>(p, p.hist, n_zero);
        {
            cudaLaunchConfig_t cfg = {};
            cfg.stream = st;
            cudaLaunchAttribute attr[1];
            attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
            attr[0].val.programmaticStreamSerializationAllowed = 1;
            cfg.attrs = attr;
            cfg.numAttrs = 1;
            cfg.gridDim = dim3(1);
            cfg.blockDim = dim3(SAMP_THREADS);
            e = cudaLaunchKernelEx(&cfg, sample_kernel<B>, p);
            if (e != cudaSuccess) return e;
            cfg.gridDim = dim3((unsigned)grid_stream);
            cfg.blockDim = dim3(256);
            if (p.U_next || p.resid) e = cudaLaunchKernelEx(&cfg, pass_kernel<B, true>, p, Q, loss_u, loss_p, u, pb, ub, sb);
            else e = cudaLaunchKernelEx(&cfg, pass_kernel<B, false>, p, Q, loss_u, loss_p, u, pb, ub, sb);
            if (e != cudaSuccess) return e;
        }
        mwu::count_launch(3);
        if (!need_p && !need_u) return cudaGetLastError();       // no threshold: every class is final
        // the list holds a few per cent of the blocks: a thread per expected entry, one CTA per SM at most.
        // Should the one-pass result be given up (once in thousands of calls), the same kernel redoes the
        // projection with the multi-pass phases.
        const long long lb = (mb / 8 + FIN_THREADS - 1) / FIN_THREADS;
        const int grid_list = (int)(lb < (long long)sm_count ? (lb > 16 ? lb : 16) : (long long)sm_count);
        return launch_cooperative(resolve_kernel<B>, grid_list, FIN_THREADS, (size_t)MP_SMEM_BYTES, sm_count, st, p, Q,
                                  loss_u, loss_p, u, pb, ub, sb);
    }
    return launch_cooperative(multipass_kernel<B>, grid_mp, FIN_THREADS, (size_t)MP_SMEM_BYTES, sm_count, st, p, Q, loss_u,
                              loss_p, u, pb, ub, sb);
}

// mwu_project and mwu_admm_step: the latter also wants U_next and / or residual_sq
static int project_impl(const mwu_proj_desc *desc, const float *W, const float *U_dual, float *Q,
                        float *U_next, double *residual_sq, float *u, uint32_t *pruned_bitmap,
                        uint32_t *unified_bitmap, uint32_t *sign_bits, double *loss_u, double *loss_p,
                        uint32_t *dev_status, void *workspace, size_t workspace_bytes, void *cuda_stream) {
    using namespace mwu;
    int rc = validate_desc(desc, false);
    if (rc != MWU_OK) return rc;
    if (!W || !u || !pruned_bitmap || !unified_bitmap || !sign_bits || !dev_status || !workspace)
        return MWU_ERR_INVALID_ARG;
    if (!aligned_to(U_next, 16) || !aligned_to(residual_sq, 8)) return MWU_ERR_ALIGNMENT;
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
    if (shape_of(desc).shaped)                          // 2- and 3-dim blocks: the block-by-block path
        return shapes::project(desc, W, U_dual, Q, U_next, residual_sq, u, pruned_bitmap, unified_bitmap, sign_bits,
                               loss_u, loss_p, dev_status, workspace, sm_count, st);
    const bool one_pass = use_one_pass(desc);
    proj::Params p;
    p.W = W;
    p.U = U_dual;
    p.n_floats = desc->rows * desc->cols;
    p.n_blocks = p.n_floats / desc->block;
    p.b = desc->block;
    p.use_l1 = desc->prune_key == MWU_PRUNE_KEY_L1;
    p.work = (proj::Work *)ws;
    p.nb = p.n_blocks <= (8ll << 20) ? proj::NB_SMALL : proj::NB_MAX;
    p.hist = (unsigned *)(ws + ws_off_hist());
    p.fhist = p.hist + 3 * (size_t)p.nb;
    p.cand_key = (proj::u64 *)(ws + ws_off_cand_key());
    p.cand_idx = (unsigned *)(ws + ws_off_cand_idx());
    p.cand_aux = (unsigned *)(ws + ws_off_cand_aux());
    p.samp_kp = (proj::u64 *)(ws + ws_off_samp());
    p.samp_ku = p.samp_kp + proj::NSAMP;
    p.bins = (unsigned *)(ws + ws_off_bins());
    p.list = (uint2 *)(ws + ws_off_list((size_t)p.n_blocks));
    p.list_cap = (unsigned)list_capacity((size_t)p.n_blocks);
    p.gated = one_pass ? 1 : 0;
    p.run_sample = one_pass ? 0 : 1;
    p.dev_status = dev_status;
    p.U_next = U_next;
    p.resid = residual_sq;
    p.k_unify = desc->k_unify;
    p.k_prune = desc->k_prune;
    p.blocks_per_row = (unsigned)(desc->cols / desc->block);
    double *gkey = nullptr;
    unsigned *gprune = nullptr;
    p.gprune = nullptr;
    p.group_rows = p.group_cols = p.groups_per_row = 1;
    if (grouped(desc)) {
        gkey = (double *)(ws + ws_off_gkey((size_t)p.n_blocks));
        gprune = (unsigned *)(ws + ws_off_gprune(desc, (size_t)p.n_blocks));
        p.gprune = gprune;
        p.group_rows = (unsigned)desc->prune_group_rows;
        p.group_cols = (unsigned)desc->prune_group_cols;
        p.groups_per_row = (unsigned)(desc->cols / desc->prune_group_cols);
    }

    // The one-pass pipeline clears its selection state and histograms in its first kernel; the
    // multi-pass kernel, launched alone, needs them (and its barrier counter) cleared beforehand.
    if (!one_pass &&
        cudaMemsetAsync(ws, 0, ws_off_hist() + 5 * (size_t)p.nb * sizeof(unsigned), st) != cudaSuccess)
        return MWU_ERR_CUDA;
    cudaError_t e;
    switch (desc->block) {
        case 2: e = launch_project<2>(p, desc, Q, u, pruned_bitmap, unified_bitmap, sign_bits, loss_u, loss_p, sm_count, one_pass, gkey, gprune, st); break;
        case 4: e = launch_project<4>(p, desc, Q, u, pruned_bitmap, unified_bitmap, sign_bits, loss_u, loss_p, sm_count, one_pass, gkey, gprune, st); break;
        case 8: e = launch_project<8>(p, desc, Q, u, pruned_bitmap, unified_bitmap, sign_bits, loss_u, loss_p, sm_count, one_pass, gkey, gprune, st); break;
        default: e = launch_project<16>(p, desc, Q, u, pruned_bitmap, unified_bitmap, sign_bits, loss_u, loss_p, sm_count, one_pass, gkey, gprune, st); break;
    }
    return e == cudaSuccess ? MWU_OK : MWU_ERR_CUDA;
}

extern "C" int mwu_project(const mwu_proj_desc *desc, const float *W, const float *U_dual, float *Q,
                           float *u, uint32_t *pruned_bitmap, uint32_t *unified_bitmap,
                           uint32_t *sign_bits, double *loss_u, double *loss_p, uint32_t *dev_status,
                           void *workspace, size_t workspace_bytes, void *cuda_stream) {
    return project_impl(desc, W, U_dual, Q, nullptr, nullptr, u, pruned_bitmap, unified_bitmap, sign_bits,
                        loss_u, loss_p, dev_status, workspace, workspace_bytes, cuda_stream);
}

extern "C" int mwu_admm_step(const mwu_proj_desc *desc, const float *W, const float *U_dual, float *Q,
                             float *U_next, double *residual_sq, float *u, uint32_t *pruned_bitmap,
                             uint32_t *unified_bitmap, uint32_t *sign_bits, uint32_t *dev_status,
                             void *workspace, size_t workspace_bytes, void *cuda_stream) {
    if (!desc || !W) return MWU_ERR_INVALID_ARG;
    if (!U_next && !residual_sq) return MWU_ERR_INVALID_ARG;       // nothing beyond mwu_project was asked for
    if (U_next) {
        // the kernels read W and U_dual again after U_next has been written: no overlap allowed
        const size_t bytes = (size_t)desc->rows * (size_t)desc->cols * sizeof(float);
        const char *o = (const char *)U_next;
        const char *ins[2] = {(const char *)W, (const char *)U_dual};
        for (int i = 0; i < 2; ++i)
            if (ins[i] && o < ins[i] + bytes && ins[i] < o + bytes) return MWU_ERR_INVALID_ARG;
    }
    return project_impl(desc, W, U_dual, Q, U_next, residual_sq, u, pruned_bitmap, unified_bitmap, sign_bits,
                        nullptr, nullptr, dev_status, workspace, workspace_bytes, cuda_stream);
}
