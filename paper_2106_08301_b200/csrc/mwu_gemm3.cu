// Decode-once path of mwu_gemm for many activation rows.
//
// The fused kernels decode a weight record again for every activation tile that meets it.  When
// the caller lends a workspace, the packed weights are instead expanded once per call into a
// row-major bf16 matrix (mwu_decode_kernel), and a plain two-operand tensor-core GEMM reads it
// (mwu_dense_pair_kernel).  The GEMM still skips what the packed format marks dead: a 64-wide
// k stage whose blocks are pruned in all 256 weight rows of a tile is neither loaded nor
// multiplied, and dead 16-wide slices of a live stage are not issued.
//
// mwu_dense_pair_kernel: a cluster of two CTAs computes a 256 x 256 tile with
// tcgen05.mma.cta_group::2; each CTA loads its own 128 activation rows and its own 128 weight
// rows of a stage by TMA (no multicast), six stages deep.  The accumulators (128 lanes x 256
// fp32 columns per CTA) are double-buffered in tensor memory, so the epilogue of a tile runs
// under the main loop of the next one.  bf16 output leaves through TMA: a warp converts 32 rows x
// 64 columns, lays them out with the 128-byte swizzle in its 4 KB of shared memory and one lane
// issues a tile store (whole 128-byte lines, clipped at the edges of Y by the tensor map).
// Roles per CTA (10 warps): warp 0 TMA producer (both CTAs' loads report their bytes straight to
// the leader's barrier, cp.async.bulk.tensor with .cta_group::2); warp 1 allocates tensor memory
// and, in the leader CTA (cluster rank 0), issues the MMAs; warps 2-9 epilogue (two per 32-lane
// quarter, 128 columns each).  The producer and issuer warps run their loops with all 32 lanes and
// elect one lane only for the TMA / MMA / commit instructions themselves: inside a lane-0 branch
// the issue of one tcgen05.mma took about 100 cycles, which left the tensor pipe idle a third of
// the time; the issuer also probes the next slot's barrier before it issues the current MMAs.
// Every wait on an mbarrier is bounded; when one runs out the kernel raises MWU_DEV_TIMEOUT,
// drains what it issued, meets its partner at a cluster barrier, frees tensor memory and returns.
#include "mwu_gemm_dev.cuh"

namespace mwu {
namespace gemm {

// ------------------------------------------------------------------------------------------
// packed records -> row-major bf16
// ------------------------------------------------------------------------------------------
constexpr int DEC_THREADS = 128;

// One CTA per 128 x 64 record: the class lists are expanded into the swizzled tile in shared
// memory exactly as the fused kernels do, then the tile is written out row by row (a warp
// writes four 128-byte row segments per instruction).  `ldw` is in elements.
template <int BW>
__global__ void __launch_bounds__(DEC_THREADS)
mwu_decode_kernel(const Params p, __nv_bfloat16 *Wd, long long ldw) {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the GEMM behind may set itself up meanwhile
    MWU_CHECK_HEADER(p);
    __shared__ __align__(1024) unsigned char tile[REC_BYTES];
    constexpr int ENT = DecodeCfg<BW, DEC_THREADS>::ENT;
    const PackedRec *recs = reinterpret_cast<const PackedRec *>(p.packed + p.off_rec);
    const long long rec = blockIdx.x;
    const long long rt = rec / p.n_stages, ks = rec % p.n_stages;
    const int tid = threadIdx.x;
    PackedRec r0, r1;
    {
        const uint4 a = __ldg(reinterpret_cast<const uint4 *>(&recs[rec]));
        const uint4 b = __ldg(reinterpret_cast<const uint4 *>(&recs[rec + 1]));
        r0.ubase = a.x; r0.dbase = a.y; r0.pbase = a.z; r0.live = a.w;
        r1.ubase = b.x; r1.dbase = b.y; r1.pbase = b.z; r1.live = b.w;
    }
    unsigned m0[ENT], m1[ENT];
    fetch_entries<BW, DEC_THREADS>(r0, r1, p, tid, m0, m1);
    write_entries<BW, DEC_THREADS>(tile, r0, r1, p, tid, m0, m1);
    asm volatile("cp.async.wait_all;" ::: "memory");
    __syncthreads();
    unsigned char *out = reinterpret_cast<unsigned char *>(Wd + (rt * kTileRows) * ldw + ks * BK);
#pragma unroll
    for (int i = 0; i < (REC_BYTES / 16) / DEC_THREADS; ++i) {
        const int q = tid + i * DEC_THREADS;                // 16-byte piece: row q / 8, piece q % 8
        const int r = q >> 3, j = q & 7;
        const uint4 v = *reinterpret_cast<const uint4 *>(tile + r * 128 + ((j ^ (r & 7)) << 4));
        *reinterpret_cast<uint4 *>(out + (size_t)r * (size_t)ldw * 2 + j * 16) = v;
    }
}

template <int BW>
static cudaError_t launch_decode_bw(const Params &p, __nv_bfloat16 *Wd, long long ldw, cudaStream_t st) {
    const long long n_rec = p.n_rec_tiles * p.n_stages;
    mwu_decode_kernel<BW><<<(unsigned)n_rec, DEC_THREADS, 0, st>>>(p, Wd, ldw);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_decode(int bw, const Params &p, __nv_bfloat16 *Wd, long long ldw, cudaStream_t st) {
    switch (bw) {
        case 2: return launch_decode_bw<2>(p, Wd, ldw, st);
        case 4: return launch_decode_bw<4>(p, Wd, ldw, st);
        case 8: return launch_decode_bw<8>(p, Wd, ldw, st);
        default: return launch_decode_bw<16>(p, Wd, ldw, st);
    }
}

// ------------------------------------------------------------------------------------------
// two-operand GEMM over the decoded weights
// ------------------------------------------------------------------------------------------
constexpr int D_STAGES = 6;
constexpr int D_EPI_WARPS = 8;
constexpr int D_MMA_WARP_B = 2 + D_EPI_WARPS;        // the second MMA issuer (the first is warp 1)
constexpr int D_THREADS = 32 * (3 + D_EPI_WARPS);
constexpr int D_A_BYTES = AH_BYTES;                  // this CTA's 128 activation rows
constexpr int D_B_BYTES = REC_BYTES;                 // this CTA's 128 weight rows
constexpr int D_STAGE_BYTES = D_A_BYTES + D_B_BYTES;
constexpr int D_BAND = 8;                            // activation row tiles per band of the tile order
constexpr int D_EPI_BUFS = 1;                        // staging buffers per epilogue warp (2 with one slot fewer measured no faster)
constexpr int D_EPI_BYTES = 4096 * D_EPI_BUFS;       // each buffer: 32 rows x 64 bf16 columns

constexpr int D_LIVE_TAB = 512;                      // live masks of all weight tiles, when they fit (short reductions)

struct DenseSmem {
    unsigned long long full[D_STAGES], empty[D_STAGES], tfull[2], tempty[2], drain[2];
    unsigned tmem_base;
    int abort;
    unsigned char live_prod[MAX_STAGES_K];
    unsigned char live_mma[MAX_STAGES_K];
    unsigned char live_mma_b[MAX_STAGES_K];              // the second MMA issuer's copy
    unsigned ho_tiles, ho_ring;                        // hand-over between the two MMA issuers
    unsigned char live_tab[D_LIVE_TAB];                // [weight tile][stage], filled once at kernel start
    unsigned short cnt_tab[D_LIVE_TAB / 4];            // [weight tile]: how many of its stages are live
};

static_assert(1024 + D_STAGES * D_STAGE_BYTES + D_EPI_WARPS * D_EPI_BYTES + sizeof(DenseSmem) <= 232448,
              "dense pair kernel: shared memory above the 227 KB a CTA may have");

__global__ void __launch_bounds__(D_THREADS, 1)
mwu_dense_pair_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_w,
                      const __grid_constant__ CUtensorMap tmap_y, const Params p) {
    if (!p.all_live) MWU_CHECK_HEADER(p);
    extern __shared__ unsigned char smem_raw[];
    unsigned char *base = reinterpret_cast<unsigned char *>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    unsigned char *sA = base;
    unsigned char *sB = base + D_STAGES * D_A_BYTES;
    unsigned char *stage_buf = sB + D_STAGES * D_B_BYTES;   // epilogue: 4 KB per warp, 1024-byte aligned
    DenseSmem *sm = reinterpret_cast<DenseSmem *>(stage_buf + D_EPI_WARPS * D_EPI_BYTES);
    const int n_stages = (int)p.n_stages;
    volatile int *abort = &sm->abort;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const unsigned rank = cluster_rank();               // 0: leader (issues the MMAs), 1: peer
    const PackedRec *recs = reinterpret_cast<const PackedRec *>(p.packed + p.off_rec);
    // 32-bit tile arithmetic (the host refuses a tile count of 2^31 or more): the MMA issuer computes
    // the next tile's position between two tiles, while the tensor pipe runs dry
    const unsigned m_tiles = (unsigned)((p.M + 255) / 256);
    const unsigned n_tiles = (unsigned)((p.n_rec_tiles + 1) / 2);
    const unsigned total_tiles = m_tiles * n_tiles;
    const unsigned pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
    // k-th tile of this CTA pair.  Tiles are dealt round-robin in an order that walks bands of
    // D_BAND activation row tiles, weight tile by weight tile: the pairs running at one time then
    // share a few weight tiles and a band of activation rows, which stay in L2.
    long long mt_ = 0, nt_ = 0;
    auto tile_of = [&](long long k, long long &mt, long long &nt) -> bool {
        const unsigned long long t64 = pair + (unsigned long long)k * n_pairs;
        if (t64 >= total_tiles) return false;
        const unsigned t = (unsigned)t64, per_band = D_BAND * n_tiles;
        const unsigned band = t / per_band, r = t - band * per_band;
        const unsigned left = m_tiles - band * D_BAND, rows = left < (unsigned)D_BAND ? left : (unsigned)D_BAND;
        const unsigned q = r / rows;
        nt = q;
        mt = band * D_BAND + (r - q * rows);
        return true;
    };

    if (threadIdx.x == 0) {
        for (int s = 0; s < D_STAGES; ++s) {
            mbar_init(smem_u32(&sm->full[s]), 1);           // leader: the bytes of both CTAs' loads
            mbar_init(smem_u32(&sm->empty[s]), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&sm->tfull[b]), 1);
            mbar_init(smem_u32(&sm->tempty[b]), 2 * D_EPI_WARPS);
        }
        mbar_init(smem_u32(&sm->drain[0]), 1);
        mbar_init(smem_u32(&sm->drain[1]), 1);
        sm->abort = 0;
        sm->ho_tiles = 0;
        sm->ho_ring = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem_alloc2(smem_u32(&sm->tmem_base), 512);
    // live mask of stage ks for tile column nt: OR over its (one or two) 128-row records
    auto live_of = [&](long long nt, int ks) -> unsigned {
        if (p.all_live) return 0xFu;
        unsigned l = __ldg(&recs[(nt * 2) * n_stages + ks].live);
        if (nt * 2 + 1 < p.n_rec_tiles) l |= __ldg(&recs[(nt * 2 + 1) * n_stages + ks].live);
        return l;
    };
    // The masks of every weight tile are read once, here, when they fit: read tile by tile they put a
    // global-memory round trip in front of every tile of the producer and of the MMA issuer, which is
    // a third of a tile's time when the reduction is only four stages long.
    const bool tab_ok = (long long)n_tiles * n_stages <= D_LIVE_TAB && n_tiles <= (unsigned)(D_LIVE_TAB / 4);
    if (tab_ok) {
        for (int i = threadIdx.x; i < (int)n_tiles * n_stages; i += blockDim.x)
            sm->live_tab[i] = (unsigned char)live_of(i / n_stages, i % n_stages);
        __syncthreads();
        for (int t = threadIdx.x; t < (int)n_tiles; t += blockDim.x) {
            unsigned cnt = 0;
            for (int ks = 0; ks < n_stages; ++ks) cnt += sm->live_tab[t * n_stages + ks] != 0;
            sm->cnt_tab[t] = (unsigned short)cnt;
        }
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                                 // both CTAs' barriers exist before any remote arrive
    tc_fence_after();
    const unsigned tmem_base = *reinterpret_cast<volatile unsigned *>(&sm->tmem_base);
    // launched with programmatic stream serialization: everything above ran while the kernel before
    // (the one that expands the weights) was still finishing; its memory is complete from here on
    asm volatile("griddepcontrol.wait;" ::: "memory");

    // the masks of tile nt: a view into the table, or a fresh copy in the role's own buffer
    auto load_live = [&](unsigned char *table, long long nt) -> const unsigned char * {
        if (tab_ok) return &sm->live_tab[nt * n_stages];
        __syncwarp();
        for (int ks = lane; ks < n_stages; ks += 32) table[ks] = (unsigned char)live_of(nt, ks);
        __syncwarp();
        return table;
    };

    if (warp == 0) {
        // ---------------- TMA producer: this CTA's halves of both operands ----------------
        // Both CTAs' loads report their bytes to the leader's barrier; the leader announces the
        // bytes of the whole pair.  (The peer's bytes may land first: the phase cannot complete
        // before the leader's own arrival, which carries the expected count.)
        int stage = 0;
        unsigned phase = 0;
        bool ok = true;
        for (long long k = 0; ok && tile_of(k, mt_, nt_); ++k) {
            const long long mt = mt_, nt = nt_;
            const unsigned char *lv = load_live(sm->live_prod, nt);
            for (int ks = 0; ks < n_stages; ++ks) {
                if (!lv[ks]) continue;
                if (!mbar_wait_spin(smem_u32(&sm->empty[stage]), phase ^ 1u, abort)) ok = false;
                if (!__all_sync(0xffffffffu, ok)) { ok = false; break; }
                if (elect_one()) {
                    const unsigned bar = mbar_addr_in_cta(smem_u32(&sm->full[stage]), 0);
                    if (rank == 0) mbar_expect_tx(smem_u32(&sm->full[stage]), 2 * D_STAGE_BYTES);
                    tma_load_2d_pair(smem_u32(sA + stage * D_A_BYTES), &tmap_x, bar, ks * BK,
                                     (int)(mt * 256 + rank * 128));
                    tma_load_2d_pair(smem_u32(sB + stage * D_B_BYTES), &tmap_w, bar, ks * BK,
                                     (int)(nt * 256 + rank * 128));
                }
                __syncwarp();
                if (++stage == D_STAGES) { stage = 0; phase ^= 1u; }
            }
        }
    } else if ((warp == 1 || warp == D_MMA_WARP_B) && rank == 0) {
        // ---------------- MMA issuers (leader): warp 1 takes the even tiles, the other the odd ones ----------------
        // A tcgen05.mma is accepted only shortly before the tensor pipe gets to it, so whatever the
        // issuing thread does between two tiles (next tile's position, the accumulator hand-over, the
        // first stage's barrier) leaves the pipe idle.  With two issuers each one does that work while
        // the other one's MMAs run; each owns one accumulator buffer.  The issuer of tile k starts on
        // its stages only once the issuer of tile k-1 has got past the barrier of its last stage (the
        // hand-over word): a wait by parity is only meaningful within one phase of the barrier, and
        // an issuer running a whole tile ahead could be two phases away from a slot's barrier.  The
        // hand-over also carries the ring position, so nobody counts the other one's stages.
        const unsigned mine = (warp == 1) ? 0u : 1u;
        bool ok = true, issued_any = false;
        const unsigned idesc = make_idesc_pair(256);
        volatile unsigned *ho_tiles = &sm->ho_tiles, *ho_ring = &sm->ho_ring;
        for (long long k = 0; ok && tile_of(k, mt_, nt_); ++k) {
            if ((unsigned)(k & 1) != mine) continue;
            const long long nt = nt_;
            const unsigned buf = mine, use_phase = (unsigned)((k >> 1) & 1);
            const unsigned char *lv = load_live(mine ? sm->live_mma_b : sm->live_mma, nt);
            if (!mbar_wait_spin(smem_u32(&sm->tempty[buf]), use_phase ^ 1u, abort)) ok = false;
            if (!__all_sync(0xffffffffu, ok)) { ok = false; break; }
            // the hand-over: tiles 0 .. k-1 have been issued
            if (*ho_tiles != (unsigned)k) {
                const long long t0 = clock64();
                unsigned polls = 0;
                while (*ho_tiles != (unsigned)k) {
                    // with a long reduction this issuer idles for a whole tile: it sleeps between looks
                    if (++polls > 64u) __nanosleep(256);
                    if (*abort) { ok = false; break; }
                    if (clock64() - t0 > WAIT_LIMIT_CYCLES) { *abort = 1; ok = false; break; }
                }
            }
            if (!__all_sync(0xffffffffu, ok)) { ok = false; break; }
            const unsigned ring = *ho_ring;                 // position in the ring of slots: 0 .. 2 * D_STAGES - 1
            int stage = (int)(ring % D_STAGES);
            unsigned phase = ring / D_STAGES;
            tc_fence_after();
            bool first = true;
            // The stage loop holds no vote and no warp barrier: every lane executes the same barrier
            // probes as one warp instruction and so takes the same decisions; what the warp does
            // between two stages has to fit into the time the MMAs of one stage take.
            for (int ks = 0; ks < n_stages; ++ks) {
                const unsigned live = lv[ks];
                if (!live) continue;
                if (!mbar_wait_spin(smem_u32(&sm->full[stage]), phase, abort)) { ok = false; break; }
                tc_fence_after();
                const unsigned long long adesc = make_desc(smem_u32(sA + stage * D_A_BYTES));
                const unsigned long long bdesc = make_desc(smem_u32(sB + stage * D_B_BYTES));
                if (elect_one()) {
#pragma unroll
                    for (int k4 = 0; k4 < 4; ++k4) {
                        if ((live >> k4) & 1u) {
                            umma2_bf16(tmem_base + buf * 256u, adesc + (unsigned long long)(k4 * 2),
                                       bdesc + (unsigned long long)(k4 * 2), idesc, first ? 0u : 1u);
                            first = false;
                        }
                    }
                    umma2_commit_both(smem_u32(&sm->empty[stage]));
                }
                first = false;
                issued_any = true;
                if (++stage == D_STAGES) { stage = 0; phase ^= 1u; }
            }
            if (!__all_sync(0xffffffffu, ok)) { ok = false; break; }
            if (lane == 0) {
                *ho_ring = (unsigned)stage + phase * D_STAGES;
                __threadfence_block();
                *ho_tiles = (unsigned)(k + 1);
            }
            if (elect_one()) {
                if (!first) {
                    umma2_commit_both(smem_u32(&sm->tfull[buf]));
                } else {
                    mbar_arrive(smem_u32(&sm->tfull[buf]));
                    mbar_arrive_cluster(smem_u32(&sm->tfull[buf]), 1);
                }
            }
            __syncwarp();
        }
        // everything this thread issued must have retired before tensor memory is freed
        if (lane == 0 && issued_any) {
            umma2_commit_local(smem_u32(&sm->drain[mine]));
            mbar_wait(smem_u32(&sm->drain[mine]), 0, abort);
        }
        __syncwarp();
    } else if (warp == 1 || warp == D_MMA_WARP_B) {
        // the peer's warp 1 only owns the tensor-memory allocation
    } else {
        // ---------------- epilogue: this CTA's 128 rows x 256 columns ----------------
        const int quarter = warp & 3;                       // TMEM lanes this warp may read
        const int chalf = (warp - 2) >> 2;                  // which 128 columns
        unsigned char *stg = stage_buf + (warp - 2) * D_EPI_BYTES;
        bool ok = true;
        for (long long k = 0; ok && tile_of(k, mt_, nt_); ++k) {
            const long long mt = mt_, nt = nt_;
            const unsigned buf = (unsigned)(k & 1), use_phase = (unsigned)((k >> 1) & 1);
            unsigned any = 0;
            if (tab_ok) any = sm->cnt_tab[nt];
            else {
                for (int ks = lane; ks < n_stages; ks += 32) any |= live_of(nt, ks);
                any = __reduce_or_sync(0xffffffffu, any);
            }
            if (!mbar_wait(smem_u32(&sm->tfull[buf]), use_phase, abort)) ok = false;
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            const long long m = mt * 256 + rank * 128 + quarter * 32 + lane;
            const unsigned trow = tmem_base + ((unsigned)(quarter * 32) << 16) + buf * 256u + (unsigned)(chalf * 128);
            const long long ncol0 = nt * 256 + chalf * 128;
            if (p.y_tma) {
                const long long mrow0 = m - lane;
                // All 128 columns go to registers first and the accumulator buffer is handed back at
                // once: the hand-over to the leader's MMA issuers crosses to the other SM for one of
                // the two CTAs, and that message queues behind this SM's outgoing store data, so the
                // buffer should not also wait for the conversion and the stores.
                unsigned v[4][32];
                if (any) {
#pragma unroll
                    for (int q = 0; q < 4; ++q) tmem_ld32_issue(trow + (unsigned)(32 * q), v[q]);
#pragma unroll
                    for (int q = 0; q < 4; ++q) tmem_ld_wait(v[q]);
                } else {
#pragma unroll
                    for (int q = 0; q < 4; ++q)
#pragma unroll
                        for (int j = 0; j < 32; ++j) v[q][j] = 0u;
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) {
                    if (rank == 0) mbar_arrive(smem_u32(&sm->tempty[buf]));
                    else mbar_arrive_cluster(smem_u32(&sm->tempty[buf]), 0);
                }
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const int c0 = 64 * h;
                    if (ncol0 + c0 >= p.N || mrow0 >= p.M) break;
                    unsigned char *sbuf = stg + (D_EPI_BUFS == 2 ? h * 4096 : 0);
                    // the last store out of this buffer has read it
                    if (lane == 0) { if (D_EPI_BUFS == 2) bulk_wait_read_1(); else bulk_wait_read(); }
                    __syncwarp();
                    // row `lane`: eight 16-byte pieces, piece j at position j ^ (lane % 8) (128-byte swizzle)
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const unsigned *src = (j < 4) ? (v[2 * h] + 8 * j) : (v[2 * h + 1] + 8 * (j - 4));
                        uint4 o;
                        __nv_bfloat162 h2;
                        h2 = __floats2bfloat162_rn(__uint_as_float(src[0]), __uint_as_float(src[1]));
                        o.x = *reinterpret_cast<unsigned *>(&h2);
                        h2 = __floats2bfloat162_rn(__uint_as_float(src[2]), __uint_as_float(src[3]));
                        o.y = *reinterpret_cast<unsigned *>(&h2);
                        h2 = __floats2bfloat162_rn(__uint_as_float(src[4]), __uint_as_float(src[5]));
                        o.z = *reinterpret_cast<unsigned *>(&h2);
                        h2 = __floats2bfloat162_rn(__uint_as_float(src[6]), __uint_as_float(src[7]));
                        o.w = *reinterpret_cast<unsigned *>(&h2);
                        *reinterpret_cast<uint4 *>(sbuf + lane * 128 + ((j ^ (lane & 7)) << 4)) = o;
                    }
                    fence_proxy_async();
                    __syncwarp();
                    if (lane == 0) {
                        tma_store_2d(&tmap_y, smem_u32(sbuf), (int)(ncol0 + c0), (int)mrow0);
                        bulk_commit();
                    }
                }
                continue;                                   // the buffer went back above
            } else {
            for (int c0 = 0; c0 < 128; c0 += 32) {
                if (ncol0 + c0 >= p.N) break;
                unsigned v[32];
                if (any) {
                    tmem_ld32(trow + (unsigned)c0, v);
                } else {
#pragma unroll
                    for (int j = 0; j < 32; ++j) v[j] = 0u;
                }
                if (p.y_fp32 || ncol0 + c0 + 32 > p.N) store_row_chunk<32>(p, m, ncol0 + c0, v);
                else store_chunk_staged(p, m - lane, lane, ncol0 + c0, v, stg);
            }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                if (rank == 0) mbar_arrive(smem_u32(&sm->tempty[buf]));
                else mbar_arrive_cluster(smem_u32(&sm->tempty[buf]), 0);
            }
        }
        if (lane == 0) bulk_wait_all();                     // this warp's tile stores are done
    }

    // teardown: nobody leaves while the other CTA may still read this one's memory or barriers
    tc_fence_before();
    __syncthreads();
    // after the barrier: a role that finished its own work early must still see a flag raised later
    if (*abort && threadIdx.x == 0) atomicOr(p.dev_status, (unsigned)MWU_DEV_TIMEOUT);
    cluster_sync_all();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc2(tmem_base, 512);
    }
}

static size_t dense_smem_bytes() {
    return 1024 + (size_t)D_STAGES * D_STAGE_BYTES + (size_t)D_EPI_WARPS * D_EPI_BYTES + sizeof(DenseSmem);
}

cudaError_t launch_dense(const CUtensorMap &tmap_x, const CUtensorMap &tmap_w, const CUtensorMap &tmap_y,
                         const Params &p, int sm_count, cudaStream_t st) {
    auto kern = mwu_dense_pair_kernel;
    const size_t smem = dense_smem_bytes();
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    const long long tiles = ((p.M + 255) / 256) * ((p.n_rec_tiles + 1) / 2);
    if (tiles >= (1ll << 31)) return cudaErrorInvalidValue;
    long long pairs = sm_count / 2;
    if (tiles < pairs) pairs = tiles;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(2 * pairs));
    cfg.blockDim = dim3(D_THREADS);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    count_launch();
    return cudaLaunchKernelEx(&cfg, kern, tmap_x, tmap_w, tmap_y, p);
}

}  // namespace gemm
}  // namespace mwu
