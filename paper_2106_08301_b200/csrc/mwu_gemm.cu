// mwu_gemm / mwu_conv_implicit: Y = X . W_hat^T on the packed weights (Section 3.2).
//
// One persistent CTA per SM works on tiles of 256 activation rows x 256 weight rows (128
// activation rows when the problem has no more).  A 64-wide k stage of the weight
// tile is decoded once into shared memory and multiplied with both 128-row halves of the
// activation tile, which halves decode work, shared-memory stores and slot hand-shakes per FLOP.
// Warp roles:
//   warp 0        producer of the activation tile (A operand, bf16, K-major, 128-byte swizzle):
//                 one thread issues one TMA load per stage (GEMM); for the convolution one extra
//                 warp per 32 tile rows gathers the im2col rows with plain loads instead.
//   warp 1        allocates tensor memory and issues tcgen05.mma (one thread), M = 128, N = 256
//                 per instruction, fp32 accumulators in TMEM (columns [0,256) for the first half
//                 of the rows, [256,512) for the second).
//   warps 2-9     epilogue: tcgen05.ld -> bf16/fp32 -> global, one warp per (half, 32 rows).
//   warps 10-..   decode the weight tile (B operand) from the packed class lists into the
//                 swizzled K-major layout the MMA reads: pruned blocks -> zeros, unified blocks
//                 -> sign . bf16(u), dense blocks -> stored bf16 values.  Three groups of six
//                 warps (four for the convolution), one per pipeline slot.  A group reads the small per-entry words of its
//                 next stage before it waits for the slot; once the slot is free it writes zeros
//                 and sign . u words with plain stores and moves dense values with cp.async.
// A 64-wide k stage whose blocks are pruned in every row of the weight tile is skipped by all
// roles (no load, no decode, no MMA); inside a live stage the MMA skips dead 16-wide slices.
// Every wait on an mbarrier is bounded; when one runs out the kernel raises MWU_DEV_TIMEOUT,
// drains what it issued, frees its tensor memory and returns.
#include "mwu_gemm_dev.cuh"

namespace mwu {
namespace gemm {

// pair kernel (two CTAs per tile), defined in mwu_gemm2.cu
bool pair_eligible(const Params &p);
cudaError_t launch_pair(int bw, const CUtensorMap &tmap, const Params &p, int sm_count, cudaStream_t st);
// decode-once path, defined in mwu_gemm3.cu
cudaError_t launch_decode(int bw, const Params &p, __nv_bfloat16 *Wd, long long ldw, cudaStream_t st);
cudaError_t launch_dense(const CUtensorMap &tmap_x, const CUtensorMap &tmap_w, const CUtensorMap &tmap_y,
                         const Params &p, int sm_count,
                         cudaStream_t st);

// ------------------------------------------------------------------------------------------
// the kernel
// ------------------------------------------------------------------------------------------
struct Smem {
    unsigned long long full[STAGES], empty[STAGES], tfull, tempty, drain;
    unsigned tmem_base;
    int abort;
    unsigned char live_prod[MAX_STAGES_K];                  // live masks of the producer's tile
    unsigned char live_mma[MAX_STAGES_K];                   // ... of the MMA issuer's tile
    unsigned char live_gather[MAX_GATHER_WARPS][MAX_STAGES_K]; // ... of each gather warp's tile
    unsigned short live_list[NDEC_GROUPS][MAX_STAGES_K];    // live stage numbers of a decode group's tile
    int n_live[NDEC_GROUPS];
};

__device__ __forceinline__ void group_bar(int group, int nthreads) {   // the threads of one decode group
    asm volatile("bar.sync %0, %1;" ::"r"(1 + group), "r"(nthreads) : "memory");
}

// MODE 0: GEMM (A by TMA), 1: convolution (A gathered).  NREC: 128-row weight records per tile.
// MT: 128-row halves of the activation tile (1 or 2).
template <int MODE, int NREC, int BW, int MT>
__global__ void __launch_bounds__(cta_threads(MODE, MT), 1)
mwu_gemm_kernel(const __grid_constant__ CUtensorMap tmap, const Params p) {
    MWU_CHECK_HEADER(p);
    constexpr int NDEC_WARPS = dec_warps(MODE);
    constexpr int NDEC_THREADS = NDEC_WARPS * 32;
    constexpr int FIRST_GATHER_WARP = first_gather_warp(MODE);
    constexpr int NGATHER_WARPS = gather_warps(MODE, MT);
    extern __shared__ unsigned char smem_raw[];
    unsigned char *base = reinterpret_cast<unsigned char *>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    constexpr int A_BYTES = MT * AH_BYTES;
    constexpr int B_BYTES = NREC * REC_BYTES;
    constexpr int BM = MT * BMH;
    unsigned char *sA = base;
    unsigned char *sB = base + STAGES * A_BYTES;
    Smem *sm = reinterpret_cast<Smem *>(sB + STAGES * B_BYTES);
    const int n_stages = (int)p.n_stages;
    // per decode group: the record table of its current tile, [NREC][n_stages + 1]
    uint4 *srec = reinterpret_cast<uint4 *>(reinterpret_cast<unsigned char *>(sm) + ((sizeof(Smem) + 15) & ~(size_t)15));
    int2 *ktab = reinterpret_cast<int2 *>(srec + (size_t)NDEC_GROUPS * NREC * (n_stages + 1));   // conv only
    int2 *ptab = ktab + (MODE ? p.K : 0);                                                        // conv, staged
    unsigned char *patch = reinterpret_cast<unsigned char *>(ptab + ((MODE && p.patch_rows) ? p.K : 0));
    volatile int *abort = &sm->abort;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const PackedRec *recs = reinterpret_cast<const PackedRec *>(p.packed + p.off_rec);
    const long long m_tiles = (p.M + BM - 1) / BM;
    const long long n_tiles = (p.n_rec_tiles + NREC - 1) / NREC;
    // tile t -> (mt, nt) with nt fastest: the CTAs of a wave share a few activation row blocks and
    // sweep the packed weights, which are the smaller operand and stay resident in L2
    const long long total_tiles = m_tiles * n_tiles;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            // one barrier per slot: the A producer(s) and the decode warps of the slot's group
            mbar_init(smem_u32(&sm->full[s]), (MODE ? NGATHER_WARPS : 1) + NDEC_WARPS);
            mbar_init(smem_u32(&sm->empty[s]), 1);
        }
        mbar_init(smem_u32(&sm->tfull), 1);
        mbar_init(smem_u32(&sm->tempty), 4 * MT);
        mbar_init(smem_u32(&sm->drain), 1);
        sm->abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (MODE) {
        for (int k = threadIdx.x; k < (int)p.K; k += blockDim.x) {
            const int c = k / (p.KH * p.KW), rem = k % (p.KH * p.KW);
            const int di = rem / p.KW - p.pad, dj = rem % p.KW - p.pad;
            ktab[k] = make_int2(c * p.H * p.W + di * p.W + dj, (di & 0xffff) | (dj << 16));
            if (p.patch_rows) {
                const int c_lo = ((k / BK) * BK) / (p.KH * p.KW);      // first channel of k's stage
                ptab[k] = make_int2((c - c_lo) * p.patch_rows * p.patch_pitch + (rem / p.KW) * p.patch_pitch + dj,
                                    rem % p.KW);
            }
        }
    }
    if (warp == 1) tmem_alloc(smem_u32(&sm->tmem_base), 512);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const unsigned tmem_base = *reinterpret_cast<volatile unsigned *>(&sm->tmem_base);

    // live mask of stage ks for weight tile nt (OR over its records)
    auto live_of = [&](long long nt, int ks) -> unsigned {
        unsigned live = 0;
#pragma unroll
        for (int q = 0; q < NREC; ++q) {
            const long long rt = nt * NREC + q;
            if (rt < p.n_rec_tiles) live |= __ldg(&recs[rt * n_stages + ks].live);
        }
        return live;
    };
    // one warp copies the live masks of tile nt into its table
    auto load_live = [&](unsigned char *table, long long nt) {
        __syncwarp();
        for (int ks = lane; ks < n_stages; ks += 32) table[ks] = (unsigned char)live_of(nt, ks);
        __syncwarp();
    };

    if (warp == 0 && MODE == 0) {
        // ---------------- TMA producer ----------------
        int stage = 0;
        unsigned phase = 0;
        bool ok = true;
        for (long long t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
            const long long mt = t / n_tiles, nt = t % n_tiles;
            load_live(sm->live_prod, nt);
            if (lane == 0) {
                for (int ks = 0; ks < n_stages; ++ks) {
                    if (!sm->live_prod[ks]) continue;
                    if (!mbar_wait(smem_u32(&sm->empty[stage]), phase ^ 1u, abort)) { ok = false; break; }
                    const unsigned bar = smem_u32(&sm->full[stage]);
                    mbar_expect_tx(bar, A_BYTES);
                    tma_load_2d(smem_u32(sA + stage * A_BYTES), &tmap, bar, ks * BK, (int)(mt * BM));
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
            }
            ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        int stage = 0;
        unsigned phase = 0, acc_phase = 0;
        bool ok = true;
        bool issued_any = false;
        bool ready = false;                                 // next slot's full barrier already seen complete
        // All 32 lanes run the loop and one elected lane issues the MMAs and commits: in a
        // lane-0 branch the issue of one tcgen05.mma took about 100 cycles.
        for (long long t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
            const long long nt = t % n_tiles;
            load_live(sm->live_mma, nt);
            const int nrec_here = (int)((p.n_rec_tiles - nt * NREC) < NREC ? (p.n_rec_tiles - nt * NREC) : NREC);
            const unsigned idesc = make_idesc(nrec_here * kTileRows);
            // the epilogue must have read the previous tile's accumulators
            if (!mbar_wait(smem_u32(&sm->tempty), acc_phase ^ 1u, abort)) ok = false;
            if (!__all_sync(0xffffffffu, ok)) { ok = false; break; }
            acc_phase ^= 1u;
            tc_fence_after();
            bool first = true;
            for (int ks = 0; ks < n_stages; ++ks) {
                const unsigned live = sm->live_mma[ks];
                if (!live) continue;
                // `ready` was probed before the previous stage's MMAs were issued
                if (!ready) {
                    if (!mbar_wait_spin(smem_u32(&sm->full[stage]), phase, abort)) ok = false;
                    if (!__all_sync(0xffffffffu, ok)) { ok = false; break; }
                }
                tc_fence_after();
                const unsigned long long adesc = make_desc(smem_u32(sA + stage * A_BYTES));
                const unsigned long long bdesc = make_desc(smem_u32(sB + stage * B_BYTES));
                const int nstage = (stage + 1 == STAGES) ? 0 : stage + 1;
                const unsigned nphase = (stage + 1 == STAGES) ? (phase ^ 1u) : phase;
                ready = __all_sync(0xffffffffu, mbar_test(smem_u32(&sm->full[nstage]), nphase));
                if (elect_one()) {
#pragma unroll
                    for (int k4 = 0; k4 < 4; ++k4) {
                        if ((live >> k4) & 1u) {
#pragma unroll
                            for (int h = 0; h < MT; ++h)
                                umma_bf16(tmem_base + (unsigned)(h * 256),
                                          adesc + (unsigned long long)(h * (AH_BYTES >> 4) + k4 * 2),
                                          bdesc + (unsigned long long)(k4 * 2), idesc, first ? 0u : 1u);
                            first = false;
                        }
                    }
                    umma_commit(smem_u32(&sm->empty[stage]));
                }
                first = false;
                issued_any = true;
                __syncwarp();
                stage = nstage;
                phase = nphase;
            }
            if (!ok) break;
            if (elect_one()) {
                if (!first) umma_commit(smem_u32(&sm->tfull));
                else mbar_arrive(smem_u32(&sm->tfull));
            }
            __syncwarp();
        }
        // everything this thread issued must have retired before tensor memory is freed
        if (lane == 0 && issued_any) {
            umma_commit(smem_u32(&sm->drain));
            mbar_wait(smem_u32(&sm->drain), 0, abort);
        }
        __syncwarp();
    } else if (warp >= 2 && warp < FIRST_DEC_WARP) {
        // ---------------- epilogue ----------------
        const int quarter = warp & 3;                       // TMEM lanes this warp may read
        const int half = (warp - 2) >> 2;                   // which 128-row half of the tile
        if (half < MT) {
            unsigned acc_phase = 0;
            bool ok = true;
            for (long long t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
                const long long mt = t / n_tiles, nt = t % n_tiles;
                unsigned any = 0;
                for (int ks = lane; ks < n_stages; ks += 32) any |= live_of(nt, ks);
                any = __reduce_or_sync(0xffffffffu, any);
                if (!mbar_wait(smem_u32(&sm->tfull), acc_phase, abort)) { ok = false; }
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                acc_phase ^= 1u;
                tc_fence_after();
                const long long m = mt * BM + half * BMH + quarter * 32 + lane;
                const int ncols_tile = (int)(((p.n_rec_tiles - nt * NREC) < NREC ? (p.n_rec_tiles - nt * NREC) : NREC) * kTileRows);
                for (int c0 = 0; c0 < ncols_tile; c0 += 32) {
                    unsigned v[32];
                    if (any) {
                        tmem_ld32(tmem_base + ((unsigned)(quarter * 32) << 16) + (unsigned)(half * 256 + c0), v);
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; ++j) v[j] = 0u;
                    }
                    const long long n0 = nt * (NREC * kTileRows) + c0;
                    if (MODE == 0) {
                        if (p.stage_epi && !p.y_fp32 && n0 + 32 <= p.N)
                            store_chunk_staged(p, m - lane, lane, n0, v,
                                               reinterpret_cast<unsigned char *>(ktab) + (warp - 2) * 2048);
                        else
                            store_row_chunk<32>(p, m, n0, v);
                    } else {
                        // NCHW output: row m = (img, oh, ow); consecutive lanes write consecutive pixels
                        if (m < p.M) {
                            const long long hw = (long long)p.OH * p.OW;
                            const long long img = m / hw, pix = m % hw;
                            for (int j = 0; j < 32; ++j) {
                                const long long o = n0 + j;
                                if (o < p.N) {
                                    const long long idx = (img * p.N + o) * hw + pix;
                                    if (p.y_fp32) reinterpret_cast<float *>(p.Y)[idx] = __uint_as_float(v[j]);
                                    else reinterpret_cast<__nv_bfloat16 *>(p.Y)[idx] = __float2bfloat16_rn(__uint_as_float(v[j]));
                                }
                            }
                        }
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&sm->tempty));
            }
        }
    } else if (warp >= FIRST_DEC_WARP && warp < FIRST_GATHER_WARP) {
        // ---------------- weight decode: one group per pipeline slot ----------------
        const int group = (warp - FIRST_DEC_WARP) / NDEC_WARPS;
        const int tid = threadIdx.x - (FIRST_DEC_WARP + group * NDEC_WARPS) * 32;
        const int gwarp = tid >> 5;
        uint4 *my_rec = srec + (size_t)group * NREC * (n_stages + 1);
        unsigned short *my_list = sm->live_list[group];
        long long seq0 = 0;                                 // live stages of all earlier tiles
        bool ok = true;
        auto rec_at = [&](int q, int ks, PackedRec *r0, PackedRec *r1) {
            const uint4 a = my_rec[q * (n_stages + 1) + ks], b = my_rec[q * (n_stages + 1) + ks + 1];
            r0->ubase = a.x; r0->dbase = a.y; r0->pbase = a.z; r0->live = a.w;
            r1->ubase = b.x; r1->dbase = b.y; r1->pbase = b.z; r1->live = b.w;
        };
        constexpr int ENT = DecodeCfg<BW, NDEC_THREADS>::ENT;
        unsigned m0[NREC][ENT], m1[NREC][ENT];
        PackedRec fr0[NREC], fr1[NREC];                     // record entries of the fetched stage
        for (long long t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
            const long long nt = t % n_tiles;
            group_bar(group, NDEC_THREADS);                               // everyone is done with the previous tables
#pragma unroll
            for (int q = 0; q < NREC; ++q) {
                const long long rt = nt * NREC + q;
                for (int ks = tid; ks <= n_stages; ks += NDEC_THREADS) {
                    uint4 v = make_uint4(0, 0, 0, 0);
                    if (rt < p.n_rec_tiles) v = __ldg(reinterpret_cast<const uint4 *>(&recs[rt * n_stages + ks]));
                    if (ks == n_stages) v.w = 0;
                    my_rec[q * (n_stages + 1) + ks] = v;
                }
            }
            group_bar(group, NDEC_THREADS);
            if (gwarp == 0) {
                // compact list of the live stages of this tile
                int n = 0;
                for (int k0 = 0; k0 < n_stages; k0 += 32) {
                    const int ks = k0 + lane;
                    unsigned l = 0;
                    if (ks < n_stages) {
                        l = my_rec[ks].w;
                        if (NREC == 2) l |= my_rec[(n_stages + 1) + ks].w;
                    }
                    const unsigned m = __ballot_sync(0xffffffffu, l != 0);
                    if (l) my_list[n + __popc(m & ((1u << lane) - 1u))] = (unsigned short)ks;
                    n += __popc(m);
                }
                if (lane == 0) sm->n_live[group] = n;
            }
            group_bar(group, NDEC_THREADS);
            const int n_live = sm->n_live[group];
            auto fetch_stage = [&](int ks) {
#pragma unroll
                for (int q = 0; q < NREC; ++q) {
                    rec_at(q, ks, &fr0[q], &fr1[q]);
                    fetch_entries<BW, NDEC_THREADS>(fr0[q], fr1[q], p, tid, m0[q], m1[q]);
                }
            };
            // this group owns the live stages whose running number is congruent to `group`
            int i = (int)((group + NDEC_GROUPS - (seq0 % NDEC_GROUPS)) % NDEC_GROUPS);
            if (i < n_live) fetch_stage(my_list[i]);
            for (; i < n_live; i += NDEC_GROUPS) {
                const long long my_seq = seq0 + i;
                const int stage = group;                    // = my_seq % STAGES
                const unsigned phase = (unsigned)((my_seq / STAGES) & 1);
                if (!mbar_wait(smem_u32(&sm->empty[stage]), phase ^ 1u, abort)) ok = false;
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
#pragma unroll
                for (int q = 0; q < NREC; ++q)
                    write_entries<BW, NDEC_THREADS>(sB + stage * B_BYTES + q * REC_BYTES, fr0[q], fr1[q], p, tid,
                                                    m0[q], m1[q]);
                // the entry words of this group's next stage travel while the copies above land
                if (i + NDEC_GROUPS < n_live) fetch_stage(my_list[i + NDEC_GROUPS]);
                asm volatile("cp.async.wait_all;" ::: "memory");
                fence_proxy_async();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&sm->full[stage]));
            }
            seq0 += n_live;
        }
    } else if (MODE == 1 && warp >= FIRST_GATHER_WARP) {
        // ---------------- im2col gather of the A tile (convolution) ----------------
        const int gw = warp - FIRST_GATHER_WARP;
        const int r = threadIdx.x - FIRST_GATHER_WARP * 32;     // row of the tile, 0 .. BM-1
        const unsigned short *X = reinterpret_cast<const unsigned short *>(p.X);
        int stage = 0;
        unsigned phase = 0;
        unsigned pcount = 0;                                     // patch buffers used so far
        bool ok = true;
        const long long hw = (long long)p.OH * p.OW;
        for (long long t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
            const long long mt = t / n_tiles, nt = t % n_tiles;
            load_live(sm->live_gather[gw], nt);
            const long long m = mt * BM + r;
            const bool row_ok = m < p.M;
            const long long img = row_ok ? m / hw : 0, pix = row_ok ? m % hw : 0;
            const int ih0 = (int)(pix / p.OW) * p.stride, iw0 = (int)(pix % p.OW) * p.stride;
            const unsigned short *xrow = X + img * (long long)p.C * p.H * p.W + (long long)ih0 * p.W + iw0;
            unsigned char *row_base = sA + (r >> 7) * AH_BYTES;  // which 128-row half
            const unsigned rr = (unsigned)(r & 127);
            if (p.patch_rows) {
                // ---- staged: copy the needed input rows of the stage's channels into shared memory
                // once (8-byte loads), then assemble the im2col rows from there.  Rows and columns are
                // addressed in padded coordinates: padded row = oh*stride + i, padded col = ow*stride + j.
                const int HP = p.H + 2 * p.pad;
                const long long m_first = mt * BM;
                const long long prow0 = (m_first / hw) * HP + ((m_first % hw) / p.OW) * p.stride;
                const int PR = p.patch_rows, PW = p.patch_pitch, QW = PW / 4;
                const int prow_r = (int)(img * HP + ih0 - prow0);
                const int tbase = prow_r * PW + iw0;
                unsigned colmask = 0;                                    // tap column j stays inside the image
                for (int j = 0; j < p.KW; ++j)
                    if ((unsigned)(iw0 + j - p.pad) < (unsigned)p.W) colmask |= 1u << j;
                if (!row_ok) colmask = 0;
                for (int ks = 0; ks < n_stages; ++ks) {
                    if (!sm->live_gather[gw][ks]) continue;
                    const int c_lo = (ks * BK) / (p.KH * p.KW);
                    int c_hi = (ks * BK + BK - 1) / (p.KH * p.KW);
                    if (c_hi > p.C - 1) c_hi = p.C - 1;
                    unsigned char *buf = patch + (size_t)(pcount & 1) * ((size_t)p.patch_nch * PR * PW * 2);
                    ++pcount;
                    for (int idx = r; idx < PR * QW; idx += NGATHER_WARPS * 32) {
                        const int pr = idx / QW, q4 = (idx % QW) * 4;
                        const long long pabs = prow0 + pr;
                        const long long pimg = pabs / HP;
                        const int ih = (int)(pabs % HP) - p.pad;
                        const bool inside = pimg < p.NIMG && (unsigned)ih < (unsigned)p.H && q4 < p.W;
                        const unsigned short *src = X + ((pimg * p.C + c_lo) * p.H + ih) * (long long)p.W + q4;
                        unsigned char *dst = buf + ((size_t)pr * PW + q4) * 2;
                        for (int c = c_lo; c <= c_hi; ++c) {
                            uint2 v = make_uint2(0, 0);
                            if (inside) v = __ldg(reinterpret_cast<const uint2 *>(src));
                            *reinterpret_cast<uint2 *>(dst) = v;
                            src += (long long)p.H * p.W;
                            dst += (size_t)PR * PW * 2;
                        }
                    }
                    asm volatile("bar.sync %0, %1;" ::"r"(1 + NDEC_GROUPS), "r"(NGATHER_WARPS * 32) : "memory");
                    if (!mbar_wait(smem_u32(&sm->empty[stage]), phase ^ 1u, abort)) ok = false;
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) break;
                    unsigned char *tile = row_base + stage * A_BYTES;
                    const int2 *tab = ptab + ks * BK;
                    const unsigned short *pb = reinterpret_cast<const unsigned short *>(buf) + tbase;
#pragma unroll 2
                    for (int c = 0; c < 8; ++c) {
                        unsigned short v[8];
#pragma unroll
                        for (int e = 0; e < 8; ++e) {
                            const int2 tb = tab[c * 8 + e];
                            v[e] = 0;
                            if ((colmask >> tb.y) & 1u) v[e] = pb[tb.x];
                        }
                        uint4 o;
                        o.x = (unsigned)v[0] | ((unsigned)v[1] << 16);
                        o.y = (unsigned)v[2] | ((unsigned)v[3] << 16);
                        o.z = (unsigned)v[4] | ((unsigned)v[5] << 16);
                        o.w = (unsigned)v[6] | ((unsigned)v[7] << 16);
                        *reinterpret_cast<uint4 *>(tile + swz(rr, (unsigned)c)) = o;
                    }
                    fence_proxy_async();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&sm->full[stage]));
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
                continue;
            }
            for (int ks = 0; ks < n_stages; ++ks) {
                if (!sm->live_gather[gw][ks]) continue;
                if (!mbar_wait(smem_u32(&sm->empty[stage]), phase ^ 1u, abort)) ok = false;
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                unsigned char *tile = row_base + stage * A_BYTES;
                const int2 *tab = ktab + ks * BK;
#pragma unroll 2
                for (int c = 0; c < 8; c += 2) {
                    // sixteen loads in flight, then two 16-byte stores
                    unsigned short v[16];
#pragma unroll
                    for (int e = 0; e < 16; ++e) {
                        const int2 tb = tab[c * 8 + e];
                        const int ih = ih0 + (int)(short)(tb.y & 0xffff), iw = iw0 + (tb.y >> 16);
                        v[e] = 0;
                        if (row_ok && (unsigned)ih < (unsigned)p.H && (unsigned)iw < (unsigned)p.W)
                            v[e] = __ldg(xrow + tb.x);
                    }
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        uint4 o;
                        o.x = (unsigned)v[h * 8 + 0] | ((unsigned)v[h * 8 + 1] << 16);
                        o.y = (unsigned)v[h * 8 + 2] | ((unsigned)v[h * 8 + 3] << 16);
                        o.z = (unsigned)v[h * 8 + 4] | ((unsigned)v[h * 8 + 5] << 16);
                        o.w = (unsigned)v[h * 8 + 6] | ((unsigned)v[h * 8 + 7] << 16);
                        *reinterpret_cast<uint4 *>(tile + swz(rr, (unsigned)(c + h))) = o;
                    }
                }
                fence_proxy_async();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&sm->full[stage]));
                if (++stage == STAGES) { stage = 0; phase ^= 1u; }
            }
        }
    }

    // teardown
    tc_fence_before();
    __syncthreads();
    // after the barrier: a role that finished its own work early must still see a flag raised later
    if (*abort && threadIdx.x == 0) atomicOr(p.dev_status, (unsigned)MWU_DEV_TIMEOUT);
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
}

// ------------------------------------------------------------------------------------------
// host
// ------------------------------------------------------------------------------------------
EncodeTiledFn get_encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) != cudaSuccess ||
            qres != cudaDriverEntryPointSuccess)
            return nullptr;
        fn = reinterpret_cast<EncodeTiledFn>(ptr);
    }
    return fn;
}

static size_t smem_bytes(int nrec, int mt, long long n_stages, long long conv_k, size_t patch_bytes = 0) {
    return 1024 + (size_t)STAGES * (mt * AH_BYTES + nrec * REC_BYTES) + ((sizeof(Smem) + 15) & ~(size_t)15) +
           (size_t)NDEC_GROUPS * nrec * (n_stages + 1) * 16 + (size_t)conv_k * sizeof(int2) +
           (patch_bytes ? (size_t)conv_k * sizeof(int2) + patch_bytes : 0);
}

template <int MODE, int NREC, int BW, int MT>
static cudaError_t launch(const CUtensorMap &tmap, const Params &p, int grid, size_t smem, cudaStream_t st) {
    auto kern = mwu_gemm_kernel<MODE, NREC, BW, MT>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    kern<<<grid, cta_threads(MODE, MT), smem, st>>>(tmap, p);
    count_launch();
    return cudaGetLastError();
}

template <int MODE, int NREC, int MT>
static cudaError_t launch_bw(int bw, const CUtensorMap &tmap, const Params &p, int grid, size_t smem, cudaStream_t st) {
    switch (bw) {
        case 2: return launch<MODE, NREC, 2, MT>(tmap, p, grid, smem, st);
        case 4: return launch<MODE, NREC, 4, MT>(tmap, p, grid, smem, st);
        case 8: return launch<MODE, NREC, 8, MT>(tmap, p, grid, smem, st);
        default: return launch<MODE, NREC, 16, MT>(tmap, p, grid, smem, st);
    }
}

static void fill_common(Params &p, const mwu_proj_desc *desc, const void *packed, void *Y, int y_dtype,
                        uint32_t *dev_status) {
    const PackedLayout L = packed_layout(desc);
    p.packed = (const unsigned char *)packed;
    p.off_rec = L.off_rec; p.off_ulist = L.off_ulist; p.off_dpos = L.off_dpos;
    p.off_dpay = L.off_dpay; p.off_ppos = L.off_ppos;
    p.n_unified = (unsigned)L.n_unified; p.n_dense = (unsigned)L.n_dense; p.n_plist = (unsigned)L.n_plist;
    p.n_rec_tiles = L.n_tiles;
    p.n_stages = L.n_stages;
    p.N = desc->rows;
    p.K = desc->cols;
    p.bw = desc->block;
    p.Y = Y;
    p.y_fp32 = y_dtype;
    p.dev_status = dev_status;
}

}  // namespace gemm
}  // namespace mwu

// Activation rows from which expanding the weights once per call beats decoding them again for
// every 512-row activation tile.
static const int64_t kDecodeOnceMinRows = 1;

static bool encode_bf16_2d(mwu::gemm::EncodeTiledFn encode, CUtensorMap *tmap, const void *ptr, int64_t inner,
                           int64_t outer, int64_t ld, int box_rows) {
    const cuuint64_t gdim[2] = {(cuuint64_t)inner, (cuuint64_t)outer};
    const cuuint64_t gstride[1] = {(cuuint64_t)ld * 2};
    const cuuint32_t box[2] = {(cuuint32_t)mwu::gemm::BK, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return encode(tmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(ptr), gdim, gstride, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

extern "C" size_t mwu_gemm_workspace_bytes(const mwu_proj_desc *desc, int64_t M) {
    if (mwu::validate_desc(desc, true) != MWU_OK || M < kDecodeOnceMinRows) return 0;
    const mwu::PackedLayout L = mwu::packed_layout(desc);
    return (size_t)L.n_pad * (size_t)desc->cols * 2;
}

extern "C" int mwu_decode(const mwu_proj_desc *desc, const void *packed, void *Wd, int64_t ldw,
                          uint32_t *dev_status, void *cuda_stream) {
    using namespace mwu;
    using namespace mwu::gemm;
    int rc = validate_desc(desc, true);
    if (rc != MWU_OK) return rc;
    if (!packed || !Wd || !dev_status) return MWU_ERR_INVALID_ARG;
    if (ldw < desc->cols) return MWU_ERR_SHAPE;
    if (!aligned_to(packed, 256) || !aligned_to(Wd, 16) || ldw % 8 != 0 || !aligned_to(dev_status, 4))
        return MWU_ERR_ALIGNMENT;
    rc = check_device(nullptr);
    if (rc != MWU_OK) return rc;
    Params p = {};
    fill_common(p, desc, packed, nullptr, 0, dev_status);
    return launch_decode(desc->block, p, (__nv_bfloat16 *)Wd, ldw, (cudaStream_t)cuda_stream) == cudaSuccess
               ? MWU_OK : MWU_ERR_CUDA;
}

extern "C" int mwu_gemm_ws(const mwu_proj_desc *desc, const void *packed, const void *X, int64_t M,
                           int64_t ldx, void *Y, int64_t ldy, int32_t y_dtype, void *workspace,
                           size_t workspace_bytes, uint32_t *dev_status, void *cuda_stream) {
    using namespace mwu;
    using namespace mwu::gemm;
    int rc = validate_desc(desc, true);
    if (rc != MWU_OK) return rc;
    if (!packed || !X || !Y || !dev_status || M < 0) return MWU_ERR_INVALID_ARG;
    if (y_dtype != 0 && y_dtype != 1) return MWU_ERR_INVALID_ARG;
    if (ldx < desc->cols || ldy < desc->rows) return MWU_ERR_SHAPE;
    if (M >= (int64_t(1) << 31) || ldx >= (int64_t(1) << 31)) return MWU_ERR_SHAPE;
    if (!aligned_to(packed, 256) || !aligned_to(X, 16) || !aligned_to(Y, 16) || ldx % 8 != 0 ||
        ldy % (y_dtype ? 4 : 8) != 0 || !aligned_to(dev_status, 4))
        return MWU_ERR_ALIGNMENT;
    if (workspace && !aligned_to(workspace, 256)) return MWU_ERR_ALIGNMENT;
    if (M == 0) return MWU_OK;
    int sm_count = 0;
    rc = check_device(&sm_count);
    if (rc != MWU_OK) return rc;
    EncodeTiledFn encode = get_encode_fn();
    if (!encode) return MWU_ERR_CUDA;
    cudaStream_t st = (cudaStream_t)cuda_stream;

    Params p = {};
    fill_common(p, desc, packed, Y, y_dtype, dev_status);
    p.M = M;
    p.ldy = ldy;
    if (p.n_stages > MAX_STAGES_K) return MWU_ERR_SHAPE;

    // decode once into the caller's workspace, then a two-operand GEMM over it
    const size_t need = mwu_gemm_workspace_bytes(desc, M);
    if (workspace && need && workspace_bytes >= need) {
        const int64_t n_pad = p.n_rec_tiles * kTileRows;
        CUtensorMap tmap_x, tmap_w;
        if (!encode_bf16_2d(encode, &tmap_x, X, desc->cols, M, ldx, BMH) ||
            !encode_bf16_2d(encode, &tmap_w, workspace, desc->cols, n_pad, desc->cols, kTileRows))
            return MWU_ERR_CUDA;
        // bf16 output leaves through TMA tile stores of 64 columns x 32 rows; fp32 output through
        // plain stores (the map is then a copy of the activation map, never used)
        CUtensorMap tmap_y = tmap_x;
        p.y_tma = 0;
        if (y_dtype == 0) {
            if (!encode_bf16_2d(encode, &tmap_y, Y, desc->rows, M, ldy, 32)) return MWU_ERR_CUDA;
            p.y_tma = 1;
        }
        if (launch_decode(desc->block, p, (__nv_bfloat16 *)workspace, desc->cols, st) != cudaSuccess)
            return MWU_ERR_CUDA;
        return launch_dense(tmap_x, tmap_w, tmap_y, p, sm_count, st) == cudaSuccess ? MWU_OK : MWU_ERR_CUDA;
    }

    // tiles of 256 activation rows unless the problem has no second half to fill
    const int mt = (M > BMH) ? 2 : 1;
    const int bm = mt * BMH;
    CUtensorMap tmap;
    if (!encode_bf16_2d(encode, &tmap, X, desc->cols, M, ldx, bm)) return MWU_ERR_CUDA;
    const int nrec = p.n_rec_tiles >= 2 ? 2 : 1;
    const long long tiles = ((M + bm - 1) / bm) * ((p.n_rec_tiles + nrec - 1) / nrec);
    const int grid = (int)(tiles < sm_count ? tiles : sm_count);
    size_t smem = smem_bytes(nrec, mt, p.n_stages, 0);
    if (smem > 227 * 1024) return MWU_ERR_SHAPE;
    cudaError_t e;
    // bf16 rows are 16-byte aligned (checked above), which the staged epilogue stores need
    if (!y_dtype && smem + NEPI_WARPS * 2048 <= 227 * 1024) {
        p.stage_epi = 1;
        smem += NEPI_WARPS * 2048;
    }
    if (mt == 2 && pair_eligible(p))
        return launch_pair(desc->block, tmap, p, sm_count, st) == cudaSuccess ? MWU_OK : MWU_ERR_CUDA;
    if (mt == 2) e = (nrec == 2) ? launch_bw<0, 2, 2>(desc->block, tmap, p, grid, smem, st)
                                 : launch_bw<0, 1, 2>(desc->block, tmap, p, grid, smem, st);
    else e = (nrec == 2) ? launch_bw<0, 2, 1>(desc->block, tmap, p, grid, smem, st)
                         : launch_bw<0, 1, 1>(desc->block, tmap, p, grid, smem, st);
    return e == cudaSuccess ? MWU_OK : MWU_ERR_CUDA;
}

extern "C" int mwu_gemm(const mwu_proj_desc *desc, const void *packed, const void *X, int64_t M,
                        int64_t ldx, void *Y, int64_t ldy, int32_t y_dtype, uint32_t *dev_status,
                        void *cuda_stream) {
    return mwu_gemm_ws(desc, packed, X, M, ldx, Y, ldy, y_dtype, nullptr, 0, dev_status, cuda_stream);
}

extern "C" int mwu_conv_implicit(const mwu_proj_desc *desc, const void *packed, const void *X_nchw,
                                 int32_t n, int32_t c, int32_t h, int32_t w, int32_t kh, int32_t kw,
                                 int32_t stride, int32_t pad, void *Y_nchw, int32_t y_dtype,
                                 uint32_t *dev_status, void *cuda_stream) {
    using namespace mwu;
    using namespace mwu::gemm;
    int rc = validate_desc(desc, true);
    if (rc != MWU_OK) return rc;
    if (!packed || !X_nchw || !Y_nchw || !dev_status) return MWU_ERR_INVALID_ARG;
    if (y_dtype != 0 && y_dtype != 1) return MWU_ERR_INVALID_ARG;
    if (n <= 0 || c <= 0 || h <= 0 || w <= 0 || kh <= 0 || kw <= 0 || stride <= 0 || pad < 0)
        return MWU_ERR_INVALID_ARG;
    if ((int64_t)c * kh * kw != desc->cols) return MWU_ERR_SHAPE;
    if (h + 2 * pad < kh || w + 2 * pad < kw || pad > 32767 || kh > 32767 || kw > 32767) return MWU_ERR_SHAPE;
    if ((int64_t)c * h * w >= (int64_t(1) << 31)) return MWU_ERR_SHAPE;
    if (!aligned_to(packed, 256) || !aligned_to(X_nchw, 16) || !aligned_to(Y_nchw, 16) ||
        !aligned_to(dev_status, 4))
        return MWU_ERR_ALIGNMENT;
    int sm_count = 0;
    rc = check_device(&sm_count);
    if (rc != MWU_OK) return rc;

    Params p = {};
    fill_common(p, desc, packed, Y_nchw, y_dtype, dev_status);
    p.X = (const __nv_bfloat16 *)X_nchw;
    p.C = c; p.H = h; p.W = w; p.KH = kh; p.KW = kw; p.stride = stride; p.pad = pad;
    p.OH = (h + 2 * pad - kh) / stride + 1;
    p.OW = (w + 2 * pad - kw) / stride + 1;
    p.M = (long long)n * p.OH * p.OW;
    p.ldy = 0;
    const int nrec = p.n_rec_tiles >= 2 ? 2 : 1;
    const int mt = (p.M > BMH) ? 2 : 1;
    p.NIMG = n;
    // staged gather: possible when image rows are 8-byte multiples and two patches fit beside the ring
    size_t patch_bytes = 0;
    if (w % 4 == 0) {
        const long long hwo = (long long)p.OH * p.OW, hp = h + 2 * pad, bm = (long long)mt * BMH;
        long long pr_max = 0;
        for (long long m0 = 0; m0 < p.M; m0 += bm) {
            const long long m1 = (m0 + bm < p.M ? m0 + bm : p.M) - 1;
            const long long r0 = (m0 / hwo) * hp + ((m0 % hwo) / p.OW) * stride;
            const long long r1 = (m1 / hwo) * hp + ((m1 % hwo) / p.OW) * stride + kh - 1;
            if (r1 - r0 + 1 > pr_max) pr_max = r1 - r0 + 1;
        }
        const int khkw = kh * kw;
        int nch = 1;
        for (long long ks = 0; ks < p.n_stages; ++ks) {
            const int c_lo = (int)(ks * BK) / khkw;
            int c_hi = (int)(ks * BK + BK - 1) / khkw;
            if (c_hi > c - 1) c_hi = c - 1;
            if (c_hi - c_lo + 1 > nch) nch = c_hi - c_lo + 1;
        }
        const size_t one = (size_t)nch * pr_max * w * 2;
        if (smem_bytes(nrec, mt, p.n_stages, desc->cols, 2 * one + 16) <= 227 * 1024 && pr_max < 32768) {
            p.patch_rows = (int)pr_max;
            p.patch_pitch = w;
            p.patch_nch = nch;
            patch_bytes = 2 * one + 16;
        }
    }
    const size_t smem = smem_bytes(nrec, mt, p.n_stages, desc->cols, patch_bytes);
    if (p.n_stages > MAX_STAGES_K || smem > 227 * 1024) return MWU_ERR_SHAPE;
    const long long tiles = ((p.M + mt * BMH - 1) / (mt * BMH)) * ((p.n_rec_tiles + nrec - 1) / nrec);
    const int grid = (int)(tiles < sm_count ? tiles : sm_count);
    CUtensorMap tmap;
    memset(&tmap, 0, sizeof(tmap));
    cudaStream_t st = (cudaStream_t)cuda_stream;
    cudaError_t e;
    if (mt == 2) e = (nrec == 2) ? launch_bw<1, 2, 2>(desc->block, tmap, p, grid, smem, st)
                                 : launch_bw<1, 1, 2>(desc->block, tmap, p, grid, smem, st);
    else e = (nrec == 2) ? launch_bw<1, 2, 1>(desc->block, tmap, p, grid, smem, st)
                         : launch_bw<1, 1, 1>(desc->block, tmap, p, grid, smem, st);
    return e == cudaSuccess ? MWU_OK : MWU_ERR_CUDA;
}
