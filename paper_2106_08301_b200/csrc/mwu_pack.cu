// mwu_pack: serialise a projection into the packed storage form (Section 3.1 / Table 1: one
// magnitude per unified block, nothing for a pruned block, one sign bit per weight).
//
//   count_kernel  one CTA per record (128 rows x 64 columns): per-row class bits, sign word,
//                 counts of unified / dense blocks and their exclusive scan over the rows.
//   scan_kernel   one CTA: exclusive scan of the per-record counts over all records, header.
//   fill_kernel   one CTA per record: writes the unified values and the bf16 payload of the
//                 dense blocks; each warp reads one row segment (256 contiguous bytes) at a time.
#include "mwu_common.cuh"

namespace mwu {
namespace pack {

struct Params {
    const float *W;
    const float *U;
    const float *u;
    const unsigned *pruned_bitmap;
    const unsigned *unified_bitmap;
    const unsigned *sign_bits;
    unsigned char *packed;
    unsigned *dev_status;
    long long rows, cols;
    int b;
    PackedLayout L;
};

struct Rec { unsigned ubase, dbase, live, zero; };
struct Meta { unsigned long long sgn; unsigned P, U; };

__global__ void __launch_bounds__(128) count_kernel(Params p) {
    const int r = threadIdx.x;
    const long long rec = blockIdx.x;
    const long long tile = rec / p.L.n_stages, stage = rec % p.L.n_stages;
    const long long n = tile * kTileRows + r;
    const int nb = kStageK / p.b;
    const unsigned mask = (nb >= 32) ? 0xffffffffu : ((1u << nb) - 1u);
    unsigned P = mask, U = 0;
    unsigned long long sgn = 0;
    if (n < p.rows) {
        const long long j0 = n * (p.cols / p.b) + stage * nb;
        P = (p.pruned_bitmap[j0 >> 5] >> (j0 & 31)) & mask;
        U = (p.unified_bitmap[j0 >> 5] >> (j0 & 31)) & mask;
        const long long f = n * p.cols + stage * kStageK;
        sgn = (unsigned long long)p.sign_bits[f >> 5] | ((unsigned long long)p.sign_bits[(f >> 5) + 1] << 32);
    }
    if (P & U) { atomicOr(p.dev_status, (unsigned)MWU_DEV_BOUNDS); U &= ~P; }
    const unsigned cu = __popc(U), cd = nb - __popc(P) - cu;
    // live 16-column slices of this row
    unsigned live = 0;
    const unsigned notP = ~P & mask;
    const int bps = (16 / p.b) > 0 ? (16 / p.b) : 1;            // blocks per 16-column slice
    for (int s = 0; s < 4; ++s) {
        const unsigned m = (p.b >= 16) ? (1u << s) : (((1u << bps) - 1u) << (s * bps));
        if (notP & m) live |= 1u << s;
    }
    // exclusive scan of (cu, cd) over the 128 rows: packed in one 32-bit word (each <= 4096)
    unsigned both = cu | (cd << 16);
    unsigned incl = both;
    const int lane = r & 31, warp = r >> 5;
    for (int off = 1; off < 32; off <<= 1) {
        const unsigned t = __shfl_up_sync(0xffffffffu, incl, off);
        if (lane >= off) incl += t;
    }
    __shared__ unsigned s_wsum[4];
    __shared__ unsigned s_live;
    if (r == 0) s_live = 0;
    if (lane == 31) s_wsum[warp] = incl;
    __syncthreads();
    unsigned base = 0;
    for (int w = 0; w < warp; ++w) base += s_wsum[w];
    const unsigned excl = base + incl - both;
    if (live) atomicOr(&s_live, live);
    __syncthreads();
    const long long rs = rec * kTileRows + r;
    Meta *meta = reinterpret_cast<Meta *>(p.packed + p.L.off_meta);
    meta[rs].sgn = sgn;
    meta[rs].P = P;
    meta[rs].U = U;
    reinterpret_cast<unsigned *>(p.packed + p.L.off_rel)[rs] = excl;     // u16 urel | u16 drel << 16
    if (r == 127) {
        const unsigned tot = excl + both;
        Rec *recs = reinterpret_cast<Rec *>(p.packed + p.L.off_rec);
        recs[rec].ubase = tot & 0xffffu;        // counts for now; scan_kernel turns them into bases
        recs[rec].dbase = tot >> 16;
        recs[rec].live = s_live;
        recs[rec].zero = 0;
    }
}

__global__ void __launch_bounds__(1024) scan_kernel(Params p) {
    const long long n_rec = p.L.n_tiles * p.L.n_stages;
    Rec *recs = reinterpret_cast<Rec *>(p.packed + p.L.off_rec);
    __shared__ unsigned long long s_u[1024], s_d[1024];
    const long long per = (n_rec + 1023) / 1024;
    const long long lo = threadIdx.x * per;
    const long long hi = (lo + per < n_rec) ? lo + per : n_rec;
    unsigned long long su = 0, sd = 0;
    for (long long i = lo; i < hi; ++i) { su += recs[i].ubase; sd += recs[i].dbase; }
    s_u[threadIdx.x] = su;
    s_d[threadIdx.x] = sd;
    __syncthreads();
    for (int off = 1; off < 1024; off <<= 1) {
        unsigned long long au = 0, ad = 0;
        if ((int)threadIdx.x >= off) { au = s_u[threadIdx.x - off]; ad = s_d[threadIdx.x - off]; }
        __syncthreads();
        s_u[threadIdx.x] += au;
        s_d[threadIdx.x] += ad;
        __syncthreads();
    }
    unsigned long long ru = s_u[threadIdx.x] - su, rd = s_d[threadIdx.x] - sd;
    for (long long i = lo; i < hi; ++i) {
        const unsigned cu = recs[i].ubase, cd = recs[i].dbase;
        recs[i].ubase = (unsigned)ru;
        recs[i].dbase = (unsigned)rd;
        ru += cu;
        rd += cd;
    }
    if (threadIdx.x == 1023) {
        if (s_u[1023] != (unsigned long long)p.L.n_unified || s_d[1023] != (unsigned long long)p.L.n_dense)
            atomicOr(p.dev_status, (unsigned)MWU_DEV_BOUNDS);
    }
    if (threadIdx.x < 32) {
        unsigned long long *h = reinterpret_cast<unsigned long long *>(p.packed);
        const unsigned long long vals[32] = {
            kMagic, 1ull, (unsigned long long)p.rows, (unsigned long long)p.cols,
            (unsigned long long)p.b, (unsigned long long)p.L.n_pad, (unsigned long long)p.L.n_tiles,
            (unsigned long long)p.L.n_stages, (unsigned long long)p.L.n_pruned,
            (unsigned long long)p.L.n_unified, (unsigned long long)p.L.n_dense,
            (unsigned long long)p.L.off_rec, (unsigned long long)p.L.off_meta,
            (unsigned long long)p.L.off_rel, (unsigned long long)p.L.off_ustream,
            (unsigned long long)p.L.off_dstream, (unsigned long long)p.L.total,
            0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0};
        h[threadIdx.x] = vals[threadIdx.x];
    }
}

__global__ void __launch_bounds__(128) fill_kernel(Params p) {
    const long long rec = blockIdx.x;
    const long long tile = rec / p.L.n_stages, stage = rec % p.L.n_stages;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const Rec *recs = reinterpret_cast<const Rec *>(p.packed + p.L.off_rec);
    const Meta *meta = reinterpret_cast<const Meta *>(p.packed + p.L.off_meta);
    const unsigned *rel = reinterpret_cast<const unsigned *>(p.packed + p.L.off_rel);
    float *ustream = reinterpret_cast<float *>(p.packed + p.L.off_ustream);
    __nv_bfloat162 *dstream = reinterpret_cast<__nv_bfloat162 *>(p.packed + p.L.off_dstream);
    const unsigned ubase = recs[rec].ubase, dbase = recs[rec].dbase;
    const int b = p.b;
    const int nb = kStageK / b;
    const unsigned mask = (nb >= 32) ? 0xffffffffu : ((1u << nb) - 1u);
    bool bad = false;
    for (int rr = 0; rr < 32; ++rr) {
        const int r = warp * 32 + rr;
        const long long n = tile * kTileRows + r;
        if (n >= p.rows) break;                       // padding rows hold nothing
        const long long rs = rec * kTileRows + r;
        const unsigned P = meta[rs].P, U = meta[rs].U;
        const unsigned D = ~P & ~U & mask;
        const unsigned rl = rel[rs];
        const unsigned long long ui0 = (unsigned long long)ubase + (rl & 0xffffu);
        const unsigned long long di0 = (unsigned long long)dbase + (rl >> 16);
        if (D) {
            const long long f = n * p.cols + stage * kStageK + 2 * lane;
            float2 v = __ldg(reinterpret_cast<const float2 *>(p.W + f));
            if (p.U) {
                const float2 d = __ldg(reinterpret_cast<const float2 *>(p.U + f));
                v.x = __fadd_rn(v.x, d.x);
                v.y = __fadd_rn(v.y, d.y);
            }
            const int i = (2 * lane) / b;             // block of this lane's pair
            if ((D >> i) & 1u) {
                const unsigned long long di = di0 + __popc(D & ((1u << i) - 1u));
                if (di < (unsigned long long)p.L.n_dense)
                    dstream[(di * b + (2 * lane - i * b)) >> 1] = __floats2bfloat162_rn(v.x, v.y);
                else
                    bad = true;
            }
        }
        if (lane < nb && ((U >> lane) & 1u)) {
            const unsigned long long ui = ui0 + __popc(U & ((1u << lane) - 1u));
            const long long j = n * (p.cols / b) + stage * nb + lane;
            if (ui < (unsigned long long)p.L.n_unified) ustream[ui] = p.u[j];
            else bad = true;
        }
    }
    if (bad) atomicOr(p.dev_status, (unsigned)MWU_DEV_BOUNDS);
}

}  // namespace pack
}  // namespace mwu

extern "C" size_t mwu_packed_bytes(const mwu_proj_desc *desc) {
    if (mwu::validate_desc(desc, true) != MWU_OK) return 0;
    return mwu::packed_layout(desc).total;
}

extern "C" int mwu_pack(const mwu_proj_desc *desc, const float *W, const float *U_dual, const float *u,
                        const uint32_t *pruned_bitmap, const uint32_t *unified_bitmap,
                        const uint32_t *sign_bits, void *packed, size_t packed_bytes,
                        uint32_t *dev_status, void *cuda_stream) {
    using namespace mwu;
    int rc = validate_desc(desc, true);
    if (rc != MWU_OK) return rc;
    if (!W || !u || !pruned_bitmap || !unified_bitmap || !sign_bits || !packed || !dev_status)
        return MWU_ERR_INVALID_ARG;
    if (!aligned_to(W, 16) || !aligned_to(U_dual, 16) || !aligned_to(u, 16) ||
        !aligned_to(pruned_bitmap, 16) || !aligned_to(unified_bitmap, 16) ||
        !aligned_to(sign_bits, 16) || !aligned_to(packed, 256) || !aligned_to(dev_status, 4))
        return MWU_ERR_ALIGNMENT;
    pack::Params p;
    p.L = packed_layout(desc);
    if (packed_bytes < p.L.total) return MWU_ERR_WORKSPACE;
    if (p.L.n_tiles * p.L.n_stages >= (int64_t(1) << 31)) return MWU_ERR_SHAPE;
    rc = check_device(nullptr);
    if (rc != MWU_OK) return rc;
    p.W = W; p.U = U_dual; p.u = u;
    p.pruned_bitmap = pruned_bitmap; p.unified_bitmap = unified_bitmap; p.sign_bits = sign_bits;
    p.packed = (unsigned char *)packed;
    p.dev_status = dev_status;
    p.rows = desc->rows; p.cols = desc->cols; p.b = desc->block;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    // gaps between sections and the tail of the last section must read as zero
    if (cudaMemsetAsync(packed, 0, kHeaderBytes, st) != cudaSuccess) return MWU_ERR_CUDA;
    const size_t gaps[5][2] = {
        {p.L.off_rec + 16 * (size_t)p.L.n_tiles * p.L.n_stages, p.L.off_meta},
        {p.L.off_meta + 16 * (size_t)p.L.n_tiles * p.L.n_stages * kTileRows, p.L.off_rel},
        {p.L.off_rel + 4 * (size_t)p.L.n_tiles * p.L.n_stages * kTileRows, p.L.off_ustream},
        {p.L.off_ustream + 4 * (size_t)p.L.n_unified, p.L.off_dstream},
        {p.L.off_dstream + 2 * (size_t)desc->block * p.L.n_dense, p.L.total}};
    for (int g = 0; g < 5; ++g)
        if (gaps[g][1] > gaps[g][0])
            if (cudaMemsetAsync((char *)packed + gaps[g][0], 0, gaps[g][1] - gaps[g][0], st) != cudaSuccess)
                return MWU_ERR_CUDA;
    const int n_rec = (int)(p.L.n_tiles * p.L.n_stages);
    pack::count_kernel<<<n_rec, 128, 0, st>>>(p);
    pack::scan_kernel<<<1, 1024, 0, st>>>(p);
    pack::fill_kernel<<<n_rec, 128, 0, st>>>(p);
    return cudaGetLastError() == cudaSuccess ? MWU_OK : MWU_ERR_CUDA;
}
