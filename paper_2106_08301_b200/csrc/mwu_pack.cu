// mwu_pack: serialise a projection into the packed storage form (Section 3.1 / Table 1: one
// magnitude per unified block, nothing but its position for a pruned block, one sign bit per
// weight of a unified block, bf16 values for the rest), arranged per GEMM tile.
//
//   count_kernel  one CTA per tile of 128 rows, a lane per record (128 rows x 64 columns) walking the
//                 rows: number of unified / dense / pruned blocks and the record's live-slice mask.
//   scan_kernel   one CTA: exclusive scan of the per-record counts over all records (1024 records
//                 at a time, read and written as whole lines), header.
//   fill_kernel   one CTA per record.  First one thread per row: class masks, then a scan over the
//                 rows of the number of blocks per (class, store slot), which gives every block its
//                 place in the round-robin order of its class list; the places go to shared memory.
//                 Then the lists leave in list order, consecutive threads writing consecutive
//                 entries; a dense block's values are read by the lanes that share its 64-byte run.
// The three are chained with programmatic stream serialization.
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
    long long bpr;                  // blocks per row: cols / b
    unsigned n_stages;              // L.n_stages, for 32-bit record arithmetic (records < 2^31)
    PackedLayout L;
    unsigned long long gap[5][2];   // byte ranges between the sections (alignment padding), zeroed by scan_kernel
};

// class masks of row r of a record; padding rows are all-pruned
__device__ __forceinline__ void row_masks(const Params &p, int nb, long long tile, long long stage, int r,
                                          unsigned *P, unsigned *U, unsigned long long *sgn) {
    const unsigned mask = (nb >= 32) ? 0xffffffffu : ((1u << nb) - 1u);
    const long long n = tile * kTileRows + r;
    *P = mask;
    *U = 0;
    *sgn = 0;
    if (n < p.rows) {
        const long long j0 = n * p.bpr + stage * nb;
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

// sign bits of one block (bit l = weight l) -> bit l/2 + 16 * (l % 2): the even bits closed up in the
// low half, the odd bits in the high half
__device__ __forceinline__ unsigned close_up_even_bits(unsigned x) {
    x &= 0x55555555u;
    x = (x | (x >> 1)) & 0x33333333u;
    x = (x | (x >> 2)) & 0x0f0f0f0fu;
    x = (x | (x >> 4)) & 0x00ff00ffu;
    x = (x | (x >> 8)) & 0x0000ffffu;
    return x;
}
__device__ __forceinline__ unsigned spread_signs(unsigned sb, int b) {
    const unsigned m = (b >= 32) ? 0xffffffffu : ((1u << b) - 1u);
    sb &= m;
    return close_up_even_bits(sb) | (close_up_even_bits(sb >> 1) << 16);
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

constexpr int COUNT_WARPS = 16;                         // each takes 8 of the tile's 128 rows

__global__ void __launch_bounds__(32 * COUNT_WARPS) count_kernel(Params p) {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const unsigned chunks = (p.n_stages + 31u) / 32u;       // 32 records of a tile at a time: lane = record (stage)
    const long long tile = blockIdx.x / chunks;
    const long long stage = (long long)(blockIdx.x % chunks) * 32 + lane;
    const int nb = kStageK / p.b;
    const unsigned mask = (nb >= 32) ? 0xffffffffu : ((1u << nb) - 1u);
    const long long bpr = p.bpr;                            // blocks per row
    constexpr int RPW = kTileRows / COUNT_WARPS;
    __shared__ unsigned s_cu[COUNT_WARPS][32], s_cp[COUNT_WARPS][32], s_live[COUNT_WARPS][32];
    unsigned cu = 0, cp = 0, live = 0;
    if (stage < p.L.n_stages) {
        unsigned P[RPW], U[RPW];
#pragma unroll
        for (int rr = 0; rr < RPW; ++rr) {                  // all of the warp's loads are in flight together
            const long long n = tile * kTileRows + warp * RPW + rr;
            P[rr] = 0xffffffffu;                            // padding rows are all-pruned
            U[rr] = 0;
            if (n < p.rows) {
                const long long j0 = n * bpr + stage * nb;
                P[rr] = __ldg(p.pruned_bitmap + (j0 >> 5)) >> (j0 & 31);
                U[rr] = __ldg(p.unified_bitmap + (j0 >> 5)) >> (j0 & 31);
            }
        }
#pragma unroll
        for (int rr = 0; rr < RPW; ++rr) {
            const unsigned Pm = P[rr] & mask;
            cu += __popc(U[rr] & mask & ~Pm);
            cp += __popc(Pm);
            live |= live_of(Pm, p.b);
        }
    }
    s_cu[warp][lane] = cu; s_cp[warp][lane] = cp; s_live[warp][lane] = live;
    __syncthreads();
    if (warp == 0 && stage < p.L.n_stages) {
        unsigned tu = 0, tp = 0, tl = 0;
#pragma unroll
        for (int w = 0; w < COUNT_WARPS; ++w) { tu += s_cu[w][lane]; tp += s_cp[w][lane]; tl |= s_live[w][lane]; }
        // counts for now (ubase, dbase, pbase, live); scan_kernel makes bases
        uint4 *recs = reinterpret_cast<uint4 *>(p.packed + p.L.off_rec);
        recs[tile * p.L.n_stages + stage] = make_uint4(tu, (unsigned)(kTileRows * nb) - tu - tp, tp, tl);
    }
}

__global__ void __launch_bounds__(1024) scan_kernel(Params p) {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const long long n_rec = p.L.n_tiles * p.L.n_stages;
    uint4 *recs = reinterpret_cast<uint4 *>(p.packed + p.L.off_rec);     // ubase, dbase, pbase, live
    __shared__ unsigned s_w[3][32];
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    asm volatile("griddepcontrol.wait;" ::: "memory");      // the counts are complete and visible
    unsigned long long cu = 0, cd = 0, cp = 0;              // totals of the chunks before this one
    constexpr int PER = 4;                                  // consecutive records per thread; a chunk is 4096 records
    for (long long g0 = 0; g0 < n_rec; g0 += PER * 1024) {
        const long long i0 = g0 + (long long)threadIdx.x * PER;
        uint4 held[PER];
        unsigned su = 0, sd = 0, sp = 0;                    // a chunk's counts fit 32 bits (at most 4096 blocks a record)
#pragma unroll
        for (int k = 0; k < PER; ++k) {
            held[k] = (i0 + k < n_rec) ? recs[i0 + k] : make_uint4(0, 0, 0, 0);
            su += held[k].x; sd += held[k].y; sp += held[k].z;
        }
        // inclusive scan of the thread sums: inside a warp, then over the 32 warp totals
        unsigned iu = su, id = sd, ip = sp;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const unsigned au = __shfl_up_sync(0xffffffffu, iu, off);
            const unsigned ad = __shfl_up_sync(0xffffffffu, id, off);
            const unsigned ap = __shfl_up_sync(0xffffffffu, ip, off);
            if (lane >= off) { iu += au; id += ad; ip += ap; }
        }
        __syncthreads();                                    // the previous chunk's warp totals have been read
        if (lane == 31) { s_w[0][wid] = iu; s_w[1][wid] = id; s_w[2][wid] = ip; }
        __syncthreads();
        unsigned wu = s_w[0][lane], wd = s_w[1][lane], wp = s_w[2][lane];     // every warp scans the 32 totals
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const unsigned au = __shfl_up_sync(0xffffffffu, wu, off);
            const unsigned ad = __shfl_up_sync(0xffffffffu, wd, off);
            const unsigned ap = __shfl_up_sync(0xffffffffu, wp, off);
            if (lane >= off) { wu += au; wd += ad; wp += ap; }
        }
        const unsigned tu = __shfl_sync(0xffffffffu, wu, 31), td = __shfl_sync(0xffffffffu, wd, 31),
                       tp = __shfl_sync(0xffffffffu, wp, 31);
        const unsigned bu = __shfl_sync(0xffffffffu, wu - s_w[0][lane], wid);  // totals of the warps before this one
        const unsigned bd = __shfl_sync(0xffffffffu, wd - s_w[1][lane], wid);
        const unsigned bp = __shfl_sync(0xffffffffu, wp - s_w[2][lane], wid);
        unsigned long long ru = cu + bu + (iu - su), rd = cd + bd + (id - sd), rp = cp + bp + (ip - sp);
#pragma unroll
        for (int k = 0; k < PER; ++k) {
            if (i0 + k < n_rec) recs[i0 + k] = make_uint4((unsigned)ru, (unsigned)rd, (unsigned)rp, held[k].w);
            ru += held[k].x; rd += held[k].y; rp += held[k].z;
        }
        cu += tu; cd += td; cp += tp;
    }
    if (threadIdx.x == 1023) {
        if (cu != (unsigned long long)p.L.n_unified || cd != (unsigned long long)p.L.n_dense ||
            cp != (unsigned long long)p.L.n_plist)
            atomicOr(p.dev_status, (unsigned)MWU_DEV_BOUNDS);
        recs[n_rec] = make_uint4((unsigned)cu, (unsigned)cd, (unsigned)cp, 0u);
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

// row and block of a tile offset (the inverse of tile_offset)
__device__ __forceinline__ void row_block_of(unsigned off, int b, unsigned *r, unsigned *i) {
    const unsigned rr = (off >> 10) * 8u + ((off >> 7) & 7u);
    const unsigned c = ((off >> 4) & 7u) ^ (rr & 7u);
    *r = rr;
    *i = (c * 16u + (off & 15u)) / (2u * (unsigned)b);
}

template <int B>
__global__ void __launch_bounds__(128) fill_kernel(Params p) {
    constexpr int NBK = kStageK / B;
    constexpr unsigned MASK = (NBK >= 32) ? 0xffffffffu : ((1u << NBK) - 1u);
    constexpr int STORE = (B >= 8) ? 16 : 2 * B;            // bytes of one shared-memory store
    constexpr int G = 128 / STORE;                          // store slots of a 128-byte row
    constexpr int LPB = (B >= 4) ? B / 4 : 1;               // lanes that share a dense block's run of W
    const unsigned rec = blockIdx.x;
    const unsigned tile_u = rec / p.n_stages;
    const long long tile = tile_u, stage = rec - tile_u * p.n_stages;
    const int r = threadIdx.x, lane = r & 31, warp = r >> 5;
    const uint4 *recs = reinterpret_cast<const uint4 *>(p.packed + p.L.off_rec);
    uint2 *ulist = reinterpret_cast<uint2 *>(p.packed + p.L.off_ulist);
    unsigned short *dpos = reinterpret_cast<unsigned short *>(p.packed + p.L.off_dpos);
    unsigned char *dpay = p.packed + p.L.off_dpay;
    unsigned short *ppos = reinterpret_cast<unsigned short *>(p.packed + p.L.off_ppos);

    __shared__ unsigned s_bal[4][3 * G];                    // per warp and (class, slot): the rows that have such a block
    __shared__ unsigned char s_before[4][3 * G];            // ... how many in the warps before
    __shared__ __align__(4) unsigned char s_len[3 * G];     // ... and in all (at most 128 each: a byte)
    __shared__ unsigned short s_full[3][kTileRows + 1];     // per class and q: list entries of rounds 0 .. q-1
    __shared__ unsigned s_more[3][kTileRows + 1];           // per class and q: slots that have a round q
    __shared__ unsigned short s_off[3][kTileRows * NBK];    // tile offsets of each class list, in list order
    unsigned P, U;
    unsigned long long sgn;
    row_masks(p, NBK, tile, stage, r, &P, &U, &sgn);
    const unsigned D = ~P & ~U & MASK;
    // class of block i: 0 pruned, 1 dense, 2 unified.  occ[class]: the store slots this row fills with it
    // (a row never has two blocks in one slot)
    unsigned occ[3] = {0u, 0u, 0u};
#pragma unroll
    for (int i = 0; i < NBK; ++i) {
        const unsigned slot = (tile_offset((unsigned)r, (unsigned)i, B) & 127u) / STORE;
        const unsigned bit = 1u << slot;
        occ[0] |= ((P >> i) & 1u) ? bit : 0u;
        occ[1] |= ((D >> i) & 1u) ? bit : 0u;
        occ[2] |= ((U >> i) & 1u) ? bit : 0u;
    }
#pragma unroll
    for (int c = 0; c < 3; ++c) {
#pragma unroll
        for (int sl = 0; sl < G; ++sl) {
            const unsigned bal = __ballot_sync(0xffffffffu, (occ[c] >> sl) & 1u);
            if (lane == ((c * G + sl) & 31)) s_bal[warp][c * G + sl] = bal;
        }
    }
    __syncthreads();
    // blocks per (class, slot) in the record, and in the warps before each warp (population counts
    // are few to a clock, so each is taken once per CTA, not once per thread)
    for (int t = r; t < 4 * 3 * G; t += kTileRows) {
        const int ww = t / (3 * G), f = t % (3 * G);
        unsigned before = 0;
        for (int w2 = 0; w2 < ww; ++w2) before += __popc(s_bal[w2][f]);
        s_before[ww][f] = (unsigned char)before;
        if (ww == 3) s_len[f] = (unsigned char)(before + __popc(s_bal[3][f]));
    }
    __syncthreads();
    // round-robin order of a class list: round q takes the q-th block of every slot that has one.
    // Thread q (and thread 0 for q = 128) tabulates what comes before round q.
    for (int q = r; q <= kTileRows; q += kTileRows) {
#pragma unroll
        for (int c = 0; c < 3; ++c) {
            // four slots at a time: bytewise minimum summed with a dot product, bytewise compare
            // gathered into a bit per slot
            unsigned full = 0, more = 0;
            const unsigned q4 = (unsigned)q * 0x01010101u;
            const unsigned *len4 = reinterpret_cast<const unsigned *>(s_len + c * G);
#pragma unroll
            for (int w = 0; w < G / 4; ++w) {
                const unsigned l4 = len4[w];
                full = __dp4a(__vminu4(l4, q4), 0x01010101u, full);
                more |= (((__vcmpgtu4(l4, q4) & 0x80808080u) * 0x00204081u) >> 28) << (4 * w);
            }
            s_full[c][q] = (unsigned short)full;
            s_more[c][q] = more;
        }
    }
    __syncthreads();

    // every block's place in its class list
    const unsigned below = (1u << lane) - 1u;
#pragma unroll 4
    for (int i = 0; i < NBK; ++i) {
        const unsigned off = tile_offset((unsigned)r, (unsigned)i, B);
        const unsigned slot = (off & 127u) / STORE;
        const unsigned cls = ((U >> i) & 1u) ? 2u : (((D >> i) & 1u) ? 1u : 0u);
        const unsigned f = cls * G + slot;
        // earlier rows with the same class and slot
        const unsigned q = s_before[warp][f] + __popc(s_bal[warp][f] & below);
        // q full rounds before it, then the lower slots of its own round
        const unsigned idx = s_full[cls][q] + __popc(s_more[cls][q] & ((1u << slot) - 1u));
        s_off[cls][idx] = (unsigned short)off;
    }
    asm volatile("griddepcontrol.wait;" ::: "memory");      // the record table holds the bases
    const uint4 me = recs[rec], nx = recs[rec + 1];         // (ubase, dbase, pbase, live); the table ends with the totals
    __syncthreads();

    bool bad = false;
    constexpr unsigned BMASK = (B >= 32) ? 0xffffffffu : ((1u << B) - 1u);
    const unsigned len_u = nx.x - me.x, len_d = nx.y - me.y, len_p = nx.z - me.z;
    // the record's three list ranges must lie inside the sections (checked once, not per entry)
    if (len_u + len_d + len_p != (unsigned)(kTileRows * NBK) ||
        (unsigned long long)me.x + len_u > (unsigned long long)p.L.n_unified ||
        (unsigned long long)me.y + len_d > (unsigned long long)p.L.n_dense ||
        (unsigned long long)me.z + len_p > (unsigned long long)p.L.n_plist)
        bad = true;                                          // the table does not describe this record
    else {
        const long long row_base = tile * kTileRows;
        const long long f_base = row_base * p.cols + stage * kStageK;          // first weight of the record
        // pruned blocks: positions only
        unsigned short *pp = ppos + me.z;
        for (unsigned t = (unsigned)r; t < len_p; t += 128u) pp[t] = s_off[0][t];
        // unified blocks: sign bits, position, magnitude
        uint2 *ul = ulist + me.x;
        const long long j_base = row_base * p.bpr + stage * NBK;
        for (unsigned t = (unsigned)r; t < len_u; t += 128u) {
            const unsigned off = s_off[2][t];
            unsigned rr, i;
            row_block_of(off, B, &rr, &i);
            const long long f = f_base + (long long)rr * p.cols + i * B;
            const unsigned sb = (__ldg(p.sign_bits + (f >> 5)) >> (f & 31)) & BMASK;
            const unsigned ub = (unsigned)__bfloat16_as_ushort(__float2bfloat16_rn(__ldg(p.u + j_base + (long long)rr * p.bpr + i)));
            ul[t] = make_uint2(spread_signs(sb, B), off | (ub << 16));
        }
        // dense blocks: position, then the values, LPB lanes to a block
        unsigned short *dp = dpos + me.y;
        for (unsigned t = (unsigned)r; t < len_d; t += 128u) dp[t] = s_off[1][t];
        unsigned char *pay = dpay + (unsigned long long)me.y * (2 * B);
        for (unsigned q = (unsigned)r; q < len_d * (unsigned)LPB; q += 128u) {
            const unsigned t = q / (unsigned)LPB, part = q % (unsigned)LPB;
            unsigned rr, i;
            row_block_of(s_off[1][t], B, &rr, &i);
            const long long f = f_base + (long long)rr * p.cols + i * B + part * 4;
            unsigned char *dst = pay + q * 8u;               // = t * 2B + part * 8 when a block takes LPB lanes
            if (B >= 4) {
                float4 a = __ldg(reinterpret_cast<const float4 *>(p.W + f));
                if (p.U) {
                    const float4 d = __ldg(reinterpret_cast<const float4 *>(p.U + f));
                    a.x = __fadd_rn(a.x, d.x); a.y = __fadd_rn(a.y, d.y); a.z = __fadd_rn(a.z, d.z); a.w = __fadd_rn(a.w, d.w);
                }
                const __nv_bfloat162 h0 = __floats2bfloat162_rn(a.x, a.y), h1 = __floats2bfloat162_rn(a.z, a.w);
                *reinterpret_cast<uint2 *>(dst) = make_uint2(*reinterpret_cast<const unsigned *>(&h0),
                                                             *reinterpret_cast<const unsigned *>(&h1));
            } else {
                float2 a = __ldg(reinterpret_cast<const float2 *>(p.W + f));
                if (p.U) {
                    const float2 d = __ldg(reinterpret_cast<const float2 *>(p.U + f));
                    a.x = __fadd_rn(a.x, d.x); a.y = __fadd_rn(a.y, d.y);
                }
                const __nv_bfloat162 h0 = __floats2bfloat162_rn(a.x, a.y);
                *reinterpret_cast<unsigned *>(pay + q * 4u) = *reinterpret_cast<const unsigned *>(&h0);
            }
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
    p.bpr = desc->cols / desc->block;
    p.n_stages = (unsigned)p.L.n_stages;
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
    pack::count_kernel<<<(unsigned)(p.L.n_tiles * ((p.L.n_stages + 31) / 32)), 32 * pack::COUNT_WARPS, 0, st>>>(p);
    // the next two start while their predecessor drains (programmatic stream serialization) and wait
    // for its memory themselves
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cfg.gridDim = dim3(1);
    cfg.blockDim = dim3(1024);
    cudaError_t e = cudaLaunchKernelEx(&cfg, pack::scan_kernel, p);
    cfg.gridDim = dim3((unsigned)n_rec);
    cfg.blockDim = dim3(128);
    if (e == cudaSuccess) {
        switch (desc->block) {
            case 2: e = cudaLaunchKernelEx(&cfg, pack::fill_kernel<2>, p); break;
            case 4: e = cudaLaunchKernelEx(&cfg, pack::fill_kernel<4>, p); break;
            case 8: e = cudaLaunchKernelEx(&cfg, pack::fill_kernel<8>, p); break;
            default: e = cudaLaunchKernelEx(&cfg, pack::fill_kernel<16>, p); break;
        }
    }
    if (e != cudaSuccess) return MWU_ERR_CUDA;
    count_launch(3);
    return cudaGetLastError() == cudaSuccess ? MWU_OK : MWU_ERR_CUDA;
}
