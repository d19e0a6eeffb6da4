// mwu_pack: serialise a projection into the packed storage form (Section 3.1 / Table 1: one
// magnitude per unified block, nothing but its position for a pruned block, one sign bit per
// weight of a unified block, bf16 values for the rest), arranged per GEMM tile.
//
//   count_kernel  one CTA per record (128 rows x 64 columns): number of unified / dense / pruned
//                 blocks and the record's live-slice mask.
//   scan_kernel   one CTA: exclusive scan of the per-record counts over all records, header.
//   fill_kernel   one CTA per record, one thread per row: class masks, then a scan over the rows
//                 of the number of blocks per (class, store slot), which gives every block its
//                 place in the round-robin order of its class list; a dense block's values are
//                 read as whole 64-byte (or shorter) runs of W and written as one bf16 vector.
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
    unsigned long long gap[5][2];   // byte ranges between the sections (alignment padding), zeroed by scan_kernel
};

// class masks of row r of a record; padding rows are all-pruned
__device__ __forceinline__ void row_masks(const Params &p, long long tile, long long stage, int r,
                                          unsigned *P, unsigned *U, unsigned long long *sgn) {
    const int nb = kStageK / p.b;
    const unsigned mask = (nb >= 32) ? 0xffffffffu : ((1u << nb) - 1u);
    const long long n = tile * kTileRows + r;
    *P = mask;
    *U = 0;
    *sgn = 0;
    if (n < p.rows) {
        const long long j0 = n * (p.cols / p.b) + stage * nb;
        *P = (p.pruned_bitmap[j0 >> 5] >> (j0 & 31)) & mask;
        *U = (p.unified_bitmap[j0 >> 5] >> (j0 & 31)) & mask & ~*P;
        const long long f = n * p.cols + stage * kStageK;
        *sgn = (unsigned long long)p.sign_bits[f >> 5] |
               ((unsigned long long)p.sign_bits[(f >> 5) + 1] << 32);
    }
}

// byte offset of block i of row r inside the record's decoded tile: rows of 128 bytes, the
// row's 16-byte chunks XOR-permuted by r % 8 (the layout the tensor-core instruction reads)
__device__ __forceinline__ unsigned tile_offset(unsigned r, unsigned i, int b) {
    const unsigned byte_in_row = i * 2u * (unsigned)b;
    const unsigned c = byte_in_row >> 4, within = byte_in_row & 15u;
    return (r >> 3) * 1024u + (r & 7u) * 128u + ((c ^ (r & 7u)) << 4) + within;
}

// sign bits of one block (bit l = weight l) -> bit l/2 + 16 * (l % 2)
__device__ __forceinline__ unsigned spread_signs(unsigned sb, int b) {
    unsigned out = 0;
    for (int l = 0; l < b; ++l) out |= ((sb >> l) & 1u) << (l / 2 + 16 * (l & 1));
    return out;
}

__device__ __forceinline__ unsigned live_of(unsigned P, int b) {
    const int nb = kStageK / b;
    const unsigned mask = (nb >= 32) ? 0xffffffffu : ((1u << nb) - 1u);
    const unsigned notP = ~P & mask;
    const int bps = (16 / b) > 0 ? (16 / b) : 1;            // blocks per 16-column slice
    unsigned live = 0;
    for (int s = 0; s < 4; ++s) {
        const unsigned m = (b >= 16) ? (1u << s) : (((1u << bps) - 1u) << (s * bps));
        if (notP & m) live |= 1u << s;
    }
    return live;
}

__global__ void __launch_bounds__(128) count_kernel(Params p) {
    const int r = threadIdx.x;
    const long long rec = blockIdx.x;
    const long long tile = rec / p.L.n_stages, stage = rec % p.L.n_stages;
    const int nb = kStageK / p.b;
    unsigned P, U;
    unsigned long long sgn;
    row_masks(p, tile, stage, r, &P, &U, &sgn);
    unsigned cu = __popc(U), cp = __popc(P);
    unsigned live = live_of(P, p.b);
    for (int m = 16; m > 0; m >>= 1) {
        cu += __shfl_xor_sync(0xffffffffu, cu, m);
        cp += __shfl_xor_sync(0xffffffffu, cp, m);
        live |= __shfl_xor_sync(0xffffffffu, live, m);
    }
    __shared__ unsigned s_cu[4], s_cp[4], s_live[4];
    if ((r & 31) == 0) { s_cu[r >> 5] = cu; s_cp[r >> 5] = cp; s_live[r >> 5] = live; }
    __syncthreads();
    if (r == 0) {
        const unsigned tu = s_cu[0] + s_cu[1] + s_cu[2] + s_cu[3];
        const unsigned tp = s_cp[0] + s_cp[1] + s_cp[2] + s_cp[3];
        PackedRec *recs = reinterpret_cast<PackedRec *>(p.packed + p.L.off_rec);
        recs[rec].ubase = tu;                         // counts for now; scan_kernel makes bases
        recs[rec].dbase = kTileRows * nb - tu - tp;
        recs[rec].pbase = tp;
        recs[rec].live = s_live[0] | s_live[1] | s_live[2] | s_live[3];
    }
}

__global__ void __launch_bounds__(1024) scan_kernel(Params p) {
    const long long n_rec = p.L.n_tiles * p.L.n_stages;
    uint4 *recs = reinterpret_cast<uint4 *>(p.packed + p.L.off_rec);     // ubase, dbase, pbase, live
    __shared__ unsigned long long s_u[64], s_d[64], s_p[64];
    const long long per = (n_rec + 1023) / 1024;
    const long long lo = threadIdx.x * per;
    const long long hi = (lo + per < n_rec) ? lo + per : n_rec;
    constexpr int KEEP = 8;                                 // records held in registers
    uint4 held[KEEP];
    unsigned long long su = 0, sd = 0, sp = 0;
#pragma unroll
    for (int k = 0; k < KEEP; ++k) {
        held[k] = make_uint4(0, 0, 0, 0);
        if (lo + k < hi) held[k] = recs[lo + k];
        su += held[k].x; sd += held[k].y; sp += held[k].z;
    }
    for (long long i = lo + KEEP; i < hi; ++i) { const uint4 v = recs[i]; su += v.x; sd += v.y; sp += v.z; }
    // inclusive scan over the 1024 threads: shuffles inside a warp, then the 32 warp totals
    unsigned long long iu = su, id = sd, ip = sp;
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const unsigned long long au = __shfl_up_sync(0xffffffffu, iu, off);
        const unsigned long long ad = __shfl_up_sync(0xffffffffu, id, off);
        const unsigned long long ap = __shfl_up_sync(0xffffffffu, ip, off);
        if (lane >= off) { iu += au; id += ad; ip += ap; }
    }
    if (lane == 31) { s_u[wid] = iu; s_d[wid] = id; s_p[wid] = ip; }
    __syncthreads();
    if (wid == 0) {
        unsigned long long wu = s_u[lane], wd = s_d[lane], wp = s_p[lane];
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const unsigned long long au = __shfl_up_sync(0xffffffffu, wu, off);
            const unsigned long long ad = __shfl_up_sync(0xffffffffu, wd, off);
            const unsigned long long ap = __shfl_up_sync(0xffffffffu, wp, off);
            if (lane >= off) { wu += au; wd += ad; wp += ap; }
        }
        s_u[32 + lane] = wu; s_d[32 + lane] = wd; s_p[32 + lane] = wp;     // inclusive warp totals
    }
    __syncthreads();
    if (wid > 0) { iu += s_u[32 + wid - 1]; id += s_d[32 + wid - 1]; ip += s_p[32 + wid - 1]; }
    unsigned long long ru = iu - su, rd = id - sd, rp = ip - sp;
#pragma unroll
    for (int k = 0; k < KEEP; ++k) {
        if (lo + k < hi) {
            recs[lo + k] = make_uint4((unsigned)ru, (unsigned)rd, (unsigned)rp, held[k].w);
            ru += held[k].x; rd += held[k].y; rp += held[k].z;
        }
    }
    for (long long i = lo + KEEP; i < hi; ++i) {
        const uint4 v = recs[i];
        recs[i] = make_uint4((unsigned)ru, (unsigned)rd, (unsigned)rp, v.w);
        ru += v.x; rd += v.y; rp += v.z;
    }
    if (threadIdx.x == 1023) {
        const unsigned long long tu = iu, td = id, tp = ip;
        if (tu != (unsigned long long)p.L.n_unified || td != (unsigned long long)p.L.n_dense ||
            tp != (unsigned long long)p.L.n_plist)
            atomicOr(p.dev_status, (unsigned)MWU_DEV_BOUNDS);
        recs[n_rec] = make_uint4((unsigned)tu, (unsigned)td, (unsigned)tp, 0u);
    }
    // the padding between the sections must read as zero (each gap is shorter than the alignment)
    for (int g = 0; g < 5; ++g)
        for (unsigned long long a = p.gap[g][0] + threadIdx.x; a < p.gap[g][1]; a += blockDim.x) p.packed[a] = 0;
    if (threadIdx.x < 32) {
        unsigned long long *h = reinterpret_cast<unsigned long long *>(p.packed);
        unsigned long long v = 0;
        switch (threadIdx.x) {
            case 0: v = kMagic; break;
            case 1: v = 4; break;
            case 2: v = (unsigned long long)p.rows; break;
            case 3: v = (unsigned long long)p.cols; break;
            case 4: v = (unsigned long long)p.b; break;
            case 5: v = (unsigned long long)p.L.n_pad; break;
            case 6: v = (unsigned long long)p.L.n_tiles; break;
            case 7: v = (unsigned long long)p.L.n_stages; break;
            case 8: v = (unsigned long long)p.L.n_pruned; break;
            case 9: v = (unsigned long long)p.L.n_unified; break;
            case 10: v = (unsigned long long)p.L.n_dense; break;
            case 11: v = (unsigned long long)p.L.n_plist; break;
            case 12: v = (unsigned long long)p.L.off_rec; break;
            case 13: v = (unsigned long long)p.L.off_ulist; break;
            case 14: v = (unsigned long long)p.L.off_dpos; break;
            case 15: v = (unsigned long long)p.L.off_dpay; break;
            case 16: v = (unsigned long long)p.L.off_ppos; break;
            case 17: v = (unsigned long long)p.L.total; break;
            default: v = 0;
        }
        h[threadIdx.x] = v;
    }
}

template <int B>
__global__ void __launch_bounds__(128) fill_kernel(Params p) {
    constexpr int NBK = kStageK / B;
    constexpr unsigned MASK = (NBK >= 32) ? 0xffffffffu : ((1u << NBK) - 1u);
    constexpr int STORE = (B >= 8) ? 16 : 2 * B;            // bytes of one shared-memory store
    constexpr int G = 128 / STORE;                          // store slots of a 128-byte row
    constexpr int NF = 3 * G;                               // (class, slot) counters, 8 bits each
    constexpr int FW = NF / 4;                              // ... packed four to a word
    const long long rec = blockIdx.x;
    const long long tile = rec / p.L.n_stages, stage = rec % p.L.n_stages;
    const int r = threadIdx.x, lane = r & 31, warp = r >> 5;
    const PackedRec *recs = reinterpret_cast<const PackedRec *>(p.packed + p.L.off_rec);
    uint2 *ulist = reinterpret_cast<uint2 *>(p.packed + p.L.off_ulist);
    unsigned short *dpos = reinterpret_cast<unsigned short *>(p.packed + p.L.off_dpos);
    unsigned char *dpay = p.packed + p.L.off_dpay;
    unsigned short *ppos = reinterpret_cast<unsigned short *>(p.packed + p.L.off_ppos);
    const unsigned long long base_of[3] = {recs[rec].pbase, recs[rec].dbase, recs[rec].ubase};

    __shared__ unsigned s_warp[4][FW];
    __shared__ unsigned char s_len[NF];                     // blocks per (class, slot) in the record
    unsigned P, U;
    unsigned long long sgn;
    row_masks(p, tile, stage, r, &P, &U, &sgn);
    const unsigned D = ~P & ~U & MASK;
    // class of block i: 0 pruned, 1 dense, 2 unified; its store slot
    unsigned fld[FW];
#pragma unroll
    for (int w = 0; w < FW; ++w) fld[w] = 0;
#pragma unroll
    for (int i = 0; i < NBK; ++i) {
        const unsigned off = tile_offset((unsigned)r, (unsigned)i, B);
        const unsigned slot = (off & 127u) / STORE;
        const unsigned cls = ((U >> i) & 1u) ? 2u : (((D >> i) & 1u) ? 1u : 0u);
        const unsigned fi = cls * G + slot;
#pragma unroll
        for (int w = 0; w < FW; ++w) fld[w] += ((fi >> 2) == (unsigned)w) ? (1u << (8 * (fi & 3u))) : 0u;
    }
    // inclusive scan over the 128 rows (a field never exceeds 128, so fields do not carry)
    unsigned inc[FW];
#pragma unroll
    for (int w = 0; w < FW; ++w) inc[w] = fld[w];
    for (int off = 1; off < 32; off <<= 1) {
#pragma unroll
        for (int w = 0; w < FW; ++w) {
            const unsigned t = __shfl_up_sync(0xffffffffu, inc[w], off);
            if (lane >= off) inc[w] += t;
        }
    }
    if (lane == 31) {
#pragma unroll
        for (int w = 0; w < FW; ++w) s_warp[warp][w] = inc[w];
    }
    __syncthreads();
    unsigned excl[FW];
#pragma unroll
    for (int w = 0; w < FW; ++w) {
        unsigned b0 = 0;
        for (int ww = 0; ww < warp; ++ww) b0 += s_warp[ww][w];
        excl[w] = b0 + inc[w] - fld[w];
    }
    if (r < NF) {
        const unsigned tot = s_warp[0][r >> 2] + s_warp[1][r >> 2] + s_warp[2][r >> 2] + s_warp[3][r >> 2];
        s_len[r] = (unsigned char)((tot >> (8 * (r & 3))) & 0xffu);
    }
    __syncthreads();

    bool bad = false;
    const long long n = tile * kTileRows + r;
    constexpr unsigned BMASK = (B >= 32) ? 0xffffffffu : ((1u << B) - 1u);
#pragma unroll 4
    for (int i = 0; i < NBK; ++i) {
        const unsigned off = tile_offset((unsigned)r, (unsigned)i, B);
        const unsigned slot = (off & 127u) / STORE;
        const unsigned cls = ((U >> i) & 1u) ? 2u : (((D >> i) & 1u) ? 1u : 0u);
        const unsigned fi = cls * G + slot;
        unsigned q = 0;                                     // earlier rows with the same class and slot
#pragma unroll
        for (int w = 0; w < FW; ++w) q += ((fi >> 2) == (unsigned)w) ? ((excl[w] >> (8 * (fi & 3u))) & 0xffu) : 0u;
        // place in the round-robin order: q full rounds before it, then the lower slots of its round
        unsigned idx = 0;
#pragma unroll
        for (int sl = 0; sl < G; ++sl) {
            const unsigned len = s_len[cls * G + sl];
            idx += (len < q ? len : q) + (((unsigned)sl < slot && len > q) ? 1u : 0u);
        }
        const unsigned long long e = base_of[cls] + idx;
        if (cls == 2u) {
            const unsigned sb = (unsigned)(sgn >> (i * B)) & BMASK;
            const long long j = n * (p.cols / B) + stage * NBK + i;
            const unsigned ub = (unsigned)__bfloat16_as_ushort(__float2bfloat16_rn(__ldg(p.u + j)));
            if (e < (unsigned long long)p.L.n_unified) ulist[e] = make_uint2(spread_signs(sb, B), off | (ub << 16));
            else bad = true;
        } else if (cls == 1u) {
            if (e < (unsigned long long)p.L.n_dense) {
                dpos[e] = (unsigned short)off;
                const long long f = n * p.cols + stage * kStageK + i * B;
                float v[B];
                if (B >= 4) {
#pragma unroll
                    for (int l = 0; l < B; l += 4) {
                        float4 a = __ldg(reinterpret_cast<const float4 *>(p.W + f + l));
                        if (p.U) {
                            const float4 d = __ldg(reinterpret_cast<const float4 *>(p.U + f + l));
                            a.x = __fadd_rn(a.x, d.x); a.y = __fadd_rn(a.y, d.y); a.z = __fadd_rn(a.z, d.z); a.w = __fadd_rn(a.w, d.w);
                        }
                        v[l] = a.x; v[(l + 1) % B] = a.y; v[(l + 2) % B] = a.z; v[(l + 3) % B] = a.w;
                    }
                } else {
                    float2 a = __ldg(reinterpret_cast<const float2 *>(p.W + f));
                    if (p.U) {
                        const float2 d = __ldg(reinterpret_cast<const float2 *>(p.U + f));
                        a.x = __fadd_rn(a.x, d.x); a.y = __fadd_rn(a.y, d.y);
                    }
                    v[0] = a.x; v[1 % B] = a.y;
                }
                unsigned w[B / 2];
#pragma unroll
                for (int l = 0; l < B / 2; ++l) {
                    const __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * l], v[2 * l + 1]);
                    w[l] = *reinterpret_cast<const unsigned *>(&h);
                }
                unsigned char *dst = dpay + e * (2 * B);
                if (B == 16) {
                    *reinterpret_cast<uint4 *>(dst) = make_uint4(w[0], w[1 % (B / 2)], w[2 % (B / 2)], w[3 % (B / 2)]);
                    *reinterpret_cast<uint4 *>(dst + 16) = make_uint4(w[4 % (B / 2)], w[5 % (B / 2)], w[6 % (B / 2)], w[7 % (B / 2)]);
                } else if (B == 8) {
                    *reinterpret_cast<uint4 *>(dst) = make_uint4(w[0], w[1 % (B / 2)], w[2 % (B / 2)], w[3 % (B / 2)]);
                } else if (B == 4) {
                    *reinterpret_cast<uint2 *>(dst) = make_uint2(w[0], w[1 % (B / 2)]);
                } else {
                    *reinterpret_cast<unsigned *>(dst) = w[0];
                }
            } else {
                bad = true;
            }
        } else {
            if (e < (unsigned long long)p.L.n_plist) ppos[e] = (unsigned short)off;
            else bad = true;
        }
    }
    if (bad) atomicOr(p.dev_status, (unsigned)MWU_DEV_BOUNDS);
}

}  // namespace pack
}  // namespace mwu

extern "C" size_t mwu_packed_bytes(const mwu_proj_desc *desc) {
    if (mwu::validate_desc(desc, true) != MWU_OK) return 0;
    // a 2-dim block shape is packed through per-row arrays, which mwu_pack builds behind the packed bytes
    const size_t extra = mwu::shape_of(desc).shaped ? mwu::shapes::lowering_bytes(desc) : 0;
    return mwu::packed_layout(desc).total + extra;
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
    if (packed_bytes < mwu_packed_bytes(desc)) return MWU_ERR_WORKSPACE;
    if (p.L.n_tiles * p.L.n_stages >= (int64_t(1) << 31)) return MWU_ERR_SHAPE;
    int sm_count = 0;
    rc = check_device(&sm_count);
    if (rc != MWU_OK) return rc;
    if (shape_of(desc).shaped) {
        // every run of `block` entries of a row becomes a 1-dim block with its block's class and magnitude
        rc = shapes::lower(desc, u, pruned_bitmap, unified_bitmap, (char *)packed + p.L.total, &u, &pruned_bitmap,
                           &unified_bitmap, sm_count, (cudaStream_t)cuda_stream);
        if (rc != MWU_OK) return rc;
    }
    p.W = W; p.U = U_dual; p.u = u;
    p.pruned_bitmap = pruned_bitmap; p.unified_bitmap = unified_bitmap; p.sign_bits = sign_bits;
    p.packed = (unsigned char *)packed;
    p.dev_status = dev_status;
    p.rows = desc->rows; p.cols = desc->cols; p.b = desc->block;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    // header and the gaps between sections must read as zero: scan_kernel writes all 32 header
    // words and clears the gaps
    const size_t n_rec = (size_t)p.L.n_tiles * p.L.n_stages;
    const size_t gaps[5][2] = {
        {p.L.off_rec + 16 * (n_rec + 1), p.L.off_ulist},
        {p.L.off_ulist + 8 * (size_t)p.L.n_unified, p.L.off_dpos},
        {p.L.off_dpos + 2 * (size_t)p.L.n_dense, p.L.off_dpay},
        {p.L.off_dpay + 2 * (size_t)desc->block * p.L.n_dense, p.L.off_ppos},
        {p.L.off_ppos + 2 * (size_t)p.L.n_plist, p.L.total}};
    for (int g = 0; g < 5; ++g) { p.gap[g][0] = gaps[g][0]; p.gap[g][1] = gaps[g][1] > gaps[g][0] ? gaps[g][1] : gaps[g][0]; }
    pack::count_kernel<<<(unsigned)n_rec, 128, 0, st>>>(p);
    pack::scan_kernel<<<1, 1024, 0, st>>>(p);
    switch (desc->block) {
        case 2: pack::fill_kernel<2><<<(unsigned)n_rec, 128, 0, st>>>(p); break;
        case 4: pack::fill_kernel<4><<<(unsigned)n_rec, 128, 0, st>>>(p); break;
        case 8: pack::fill_kernel<8><<<(unsigned)n_rec, 128, 0, st>>>(p); break;
        default: pack::fill_kernel<16><<<(unsigned)n_rec, 128, 0, st>>>(p); break;
    }
    count_launch(3);
    return cudaGetLastError() == cudaSuccess ? MWU_OK : MWU_ERR_CUDA;
}
