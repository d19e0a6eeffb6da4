// Pair kernel of mwu_gemm: two CTAs of a cluster work on one tile of 512 activation rows x 256
// weight rows with tcgen05.mma.cta_group::2 (M = 256 per instruction, 128 rows in each CTA).
//
// Each CTA streams its own 256 activation rows (one TMA load per stage) and decodes only its own
// 128-row record of the weight tile; the tensor cores of both SMs read the two halves of the
// weight stage from the two shared memories.  Per FLOP this halves the decode work, the decode
// stores and the weight-operand reads of a CTA compared with the single-CTA kernel.
//
// Roles per CTA (26 warps): warp 0 TMA producer; warp 1 allocates tensor memory, and issues the
// MMAs in the leader CTA (cluster rank 0) or, in the peer, forwards "activation stage landed" to
// the leader; warps 2-9 epilogue; warps 10-25 decode, four groups of four warps, one per slot.
// Barriers: the leader's full[s] collects its own TMA, its own decode warps, the peer's decode
// warps and the peer's forwarder; tcgen05.commit with cluster multicast releases empty[s] and
// signals the accumulators (tfull) in both CTAs; the peer's epilogue warps report to the leader's
// tempty.  No TMA load uses multicast; each CTA fetches its own operands.
// Every wait is bounded as in the single-CTA kernel; the two CTAs meet at a cluster barrier before
// tensor memory is released, so neither leaves while the other can still touch its memory.
#include "mwu_gemm_dev.cuh"

namespace mwu {
namespace gemm {

constexpr int P_STAGES = 4;
constexpr int P_GROUPS = P_STAGES;
constexpr int P_DEC_WARPS = 4;
constexpr int P_DEC_THREADS = P_DEC_WARPS * 32;
constexpr int P_FIRST_DEC_WARP = 2 + NEPI_WARPS;
constexpr int P_THREADS = 32 * (P_FIRST_DEC_WARP + P_DEC_WARPS * P_GROUPS);
constexpr int P_A_BYTES = 2 * AH_BYTES;              // 256 rows of this CTA
constexpr int P_B_BYTES = REC_BYTES;                 // this CTA's 128 weight rows

struct PairSmem {
    unsigned long long full[P_STAGES], a_full[P_STAGES], empty[P_STAGES], tfull, tempty, drain;
    unsigned tmem_base;
    int abort;
    unsigned char live_prod[MAX_STAGES_K];
    unsigned char live_mma[MAX_STAGES_K];
    unsigned short live_list[P_GROUPS][MAX_STAGES_K];
    int n_live[P_GROUPS];
};

__device__ __forceinline__ void pair_group_bar(int group) {
    asm volatile("bar.sync %0, %1;" ::"r"(1 + group), "r"(P_DEC_THREADS) : "memory");
}

template <int BW>
__global__ void __launch_bounds__(P_THREADS, 1)
mwu_gemm_pair_kernel(const __grid_constant__ CUtensorMap tmap, const Params p) {
    MWU_CHECK_HEADER(p);
    extern __shared__ unsigned char smem_raw[];
    unsigned char *base = reinterpret_cast<unsigned char *>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    unsigned char *sA = base;
    unsigned char *sB = base + P_STAGES * P_A_BYTES;
    PairSmem *sm = reinterpret_cast<PairSmem *>(sB + P_STAGES * P_B_BYTES);
    const int n_stages = (int)p.n_stages;
    uint4 *srec = reinterpret_cast<uint4 *>(reinterpret_cast<unsigned char *>(sm) + ((sizeof(PairSmem) + 15) & ~(size_t)15));
    unsigned char *stage_buf = reinterpret_cast<unsigned char *>(srec + (size_t)P_GROUPS * 2 * (n_stages + 1));  // epilogue
    volatile int *abort = &sm->abort;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const unsigned rank = cluster_rank();               // 0: leader (issues the MMAs), 1: peer
    const PackedRec *recs = reinterpret_cast<const PackedRec *>(p.packed + p.off_rec);
    const long long m_tiles = (p.M + 511) / 512;
    const long long n_tiles = p.n_rec_tiles / 2;        // the host only takes this path for even counts
    const long long total_tiles = m_tiles * n_tiles;
    const long long pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
    // k-th tile of this CTA pair.  Normally tiles are dealt round-robin with the weight tile
    // fastest.  In resident mode (the whole reduction fits the pipeline slots) a pair keeps one
    // weight tile and walks the activation tiles, so the decoded weights stay in shared memory.
    auto tile_of = [&](long long k, long long &mt, long long &nt) -> bool {
        if (p.resident) {
            nt = pair % n_tiles;
            mt = pair / n_tiles + k * (n_pairs / n_tiles);
            return mt < m_tiles;
        }
        const long long t = pair + k * n_pairs;
        mt = t / n_tiles;
        nt = t % n_tiles;
        return t < total_tiles;
    };

    if (threadIdx.x == 0) {
        for (int s = 0; s < P_STAGES; ++s) {
            // leader: own TMA + own decode warps + peer decode warps + peer forwarder
            mbar_init(smem_u32(&sm->full[s]), 1 + P_DEC_WARPS + P_DEC_WARPS + 1);
            mbar_init(smem_u32(&sm->a_full[s]), 1);
            mbar_init(smem_u32(&sm->empty[s]), 1);
        }
        mbar_init(smem_u32(&sm->tfull), 1);
        mbar_init(smem_u32(&sm->tempty), 2 * NEPI_WARPS);
        mbar_init(smem_u32(&sm->drain), 1);
        sm->abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem_alloc2(smem_u32(&sm->tmem_base), 512);
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                                 // both CTAs' barriers exist before any remote arrive
    tc_fence_after();
    const unsigned tmem_base = *reinterpret_cast<volatile unsigned *>(&sm->tmem_base);

    // live mask of stage ks for pair tile nt: OR over the records of both CTAs
    auto live_of = [&](long long nt, int ks) -> unsigned {
        return __ldg(&recs[(nt * 2) * n_stages + ks].live) | __ldg(&recs[(nt * 2 + 1) * n_stages + ks].live);
    };
    auto load_live = [&](unsigned char *table, long long nt) {
        __syncwarp();
        for (int ks = lane; ks < n_stages; ks += 32) table[ks] = (unsigned char)live_of(nt, ks);
        __syncwarp();
    };

    if (warp == 0) {
        // ---------------- TMA producer: this CTA's 256 activation rows ----------------
        int stage = 0;
        unsigned phase = 0;
        bool ok = true;
        long long mt = 0, nt = 0;
        for (long long kt = 0; ok && tile_of(kt, mt, nt); ++kt) {
            load_live(sm->live_prod, nt);
            if (lane == 0) {
                for (int ks = 0; ks < n_stages; ++ks) {
                    if (!sm->live_prod[ks]) continue;
                    if (!mbar_wait(smem_u32(&sm->empty[stage]), phase ^ 1u, abort)) { ok = false; break; }
                    // the leader's loads complete on the MMA's barrier, the peer's on a local one
                    const unsigned bar = smem_u32(rank == 0 ? &sm->full[stage] : &sm->a_full[stage]);
                    mbar_expect_tx(bar, P_A_BYTES);
                    tma_load_2d(smem_u32(sA + stage * P_A_BYTES), &tmap, bar, ks * BK,
                                (int)(mt * 512 + rank * 256));
                    if (++stage == P_STAGES) { stage = 0; phase ^= 1u; }
                }
            }
            ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        }
    } else if (warp == 1 && rank == 0) {
        // ---------------- MMA issuer (leader) ----------------
        int stage = 0;
        unsigned phase = 0, acc_phase = 0;
        bool ok = true, issued_any = false, ready = false;
        const unsigned idesc = make_idesc_pair(256);
        long long mt = 0, nt = 0;
        // All 32 lanes run the loop and one elected lane issues the MMAs and commits: in a
        // lane-0 branch the issue of one tcgen05.mma took about 100 cycles.
        for (long long kt = 0; ok && tile_of(kt, mt, nt); ++kt) {
            load_live(sm->live_mma, nt);
            if (!mbar_wait(smem_u32(&sm->tempty), acc_phase ^ 1u, abort)) ok = false;
            if (!__all_sync(0xffffffffu, ok)) { ok = false; break; }
            acc_phase ^= 1u;
            tc_fence_after();
            bool first = true;
            for (int ks = 0; ks < n_stages; ++ks) {
                const unsigned live = sm->live_mma[ks];
                if (!live) continue;
                if (!ready) {
                    if (!mbar_wait_spin(smem_u32(&sm->full[stage]), phase, abort)) ok = false;
                    if (!__all_sync(0xffffffffu, ok)) { ok = false; break; }
                }
                tc_fence_after();
                const unsigned long long adesc = make_desc(smem_u32(sA + stage * P_A_BYTES));
                const unsigned long long bdesc = make_desc(smem_u32(sB + stage * P_B_BYTES));
                const int nstage = (stage + 1 == P_STAGES) ? 0 : stage + 1;
                const unsigned nphase = (stage + 1 == P_STAGES) ? (phase ^ 1u) : phase;
                ready = __all_sync(0xffffffffu, mbar_test(smem_u32(&sm->full[nstage]), nphase));
                if (elect_one()) {
#pragma unroll
                    for (int k4 = 0; k4 < 4; ++k4) {
                        if ((live >> k4) & 1u) {
#pragma unroll
                            for (int h = 0; h < 2; ++h)
                                umma2_bf16(tmem_base + (unsigned)(h * 256),
                                           adesc + (unsigned long long)(h * (AH_BYTES >> 4) + k4 * 2),
                                           bdesc + (unsigned long long)(k4 * 2), idesc, first ? 0u : 1u);
                            first = false;
                        }
                    }
                    umma2_commit_both(smem_u32(&sm->empty[stage]));
                }
                first = false;
                issued_any = true;
                __syncwarp();
                stage = nstage;
                phase = nphase;
            }
            if (!ok) break;
            if (elect_one()) {
                if (!first) {
                    umma2_commit_both(smem_u32(&sm->tfull));
                } else {
                    mbar_arrive(smem_u32(&sm->tfull));
                    mbar_arrive_cluster(smem_u32(&sm->tfull), 1);
                }
            }
            __syncwarp();
        }
        if (lane == 0 && issued_any) {
            umma2_commit_local(smem_u32(&sm->drain));
            mbar_wait(smem_u32(&sm->drain), 0, abort);
        }
        __syncwarp();
    } else if (warp == 1) {
        // ---------------- forwarder (peer): tells the leader that an activation stage landed ----------------
        int stage = 0;
        unsigned phase = 0;
        bool ok = true;
        long long mt = 0, nt = 0;
        for (long long kt = 0; ok && tile_of(kt, mt, nt); ++kt) {
            load_live(sm->live_mma, nt);
            if (lane == 0) {
                for (int ks = 0; ks < n_stages; ++ks) {
                    if (!sm->live_mma[ks]) continue;
                    if (!mbar_wait(smem_u32(&sm->a_full[stage]), phase, abort)) { ok = false; break; }
                    mbar_arrive_cluster(smem_u32(&sm->full[stage]), 0);
                    if (++stage == P_STAGES) { stage = 0; phase ^= 1u; }
                }
            }
            ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        }
    } else if (warp >= 2 && warp < P_FIRST_DEC_WARP) {
        // ---------------- epilogue: this CTA's 256 rows x 256 columns ----------------
        const int quarter = warp & 3;
        const int half = (warp - 2) >> 2;
        unsigned acc_phase = 0;
        bool ok = true;
        long long mt = 0, nt = 0;
        for (long long kt = 0; ok && tile_of(kt, mt, nt); ++kt) {
            unsigned any = 0;
            for (int ks = lane; ks < n_stages; ks += 32) any |= live_of(nt, ks);
            any = __reduce_or_sync(0xffffffffu, any);
            if (!mbar_wait(smem_u32(&sm->tfull), acc_phase, abort)) { ok = false; }
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            acc_phase ^= 1u;
            tc_fence_after();
            const long long m = mt * 512 + rank * 256 + half * BMH + quarter * 32 + lane;
            const unsigned trow = tmem_base + ((unsigned)(quarter * 32) << 16) + (unsigned)(half * 256);
            const long long ncol0 = nt * 256;
            unsigned char *stg = stage_buf + (warp - 2) * 2048;        // this warp's 32 x 64-byte buffer
            for (int c0 = 0; c0 < 256; c0 += 32) {
                unsigned v[32];
                if (any) {
                    tmem_ld32(trow + (unsigned)c0, v);
                } else {
#pragma unroll
                    for (int j = 0; j < 32; ++j) v[j] = 0u;
                }
                if (p.y_fp32 || ncol0 + c0 + 32 > p.N) {
                    store_row_chunk<32>(p, m, ncol0 + c0, v);
                    continue;
                }
                store_chunk_staged(p, m - lane, lane, ncol0 + c0, v, stg);
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                if (rank == 0) mbar_arrive(smem_u32(&sm->tempty));
                else mbar_arrive_cluster(smem_u32(&sm->tempty), 0);
            }
        }
    } else {
        // ---------------- weight decode: this CTA's record, one group per pipeline slot ----------------
        const int group = (warp - P_FIRST_DEC_WARP) / P_DEC_WARPS;
        const int tid = threadIdx.x - (P_FIRST_DEC_WARP + group * P_DEC_WARPS) * 32;
        const int gwarp = tid >> 5;
        uint4 *my_rec = srec + (size_t)group * 2 * (n_stages + 1);   // [own | other][n_stages + 1]
        unsigned short *my_list = sm->live_list[group];
        long long seq0 = 0, prev_nt = -1;
        int prev_live = -1;
        bool ok = true;
        constexpr int ENT = DecodeCfg<BW, P_DEC_THREADS>::ENT;
        unsigned m0[ENT], m1[ENT];
        PackedRec fr0, fr1;
        auto rec_at = [&](int ks, PackedRec *r0, PackedRec *r1) {
            const uint4 a = my_rec[ks], b = my_rec[ks + 1];
            r0->ubase = a.x; r0->dbase = a.y; r0->pbase = a.z; r0->live = a.w;
            r1->ubase = b.x; r1->dbase = b.y; r1->pbase = b.z; r1->live = b.w;
        };
        long long mt = 0, nt = 0;
        for (long long kt = 0; ok && tile_of(kt, mt, nt); ++kt) {
            if (p.resident && nt == prev_nt && prev_live == P_STAGES) {
                // the slots already hold this weight tile's stages (stage i sits in slot i):
                // only keep the barrier phases moving
                const int i = group;
                const long long my_seq = seq0 + i;
                const unsigned phase = (unsigned)((my_seq / P_STAGES) & 1);
                if (!mbar_wait(smem_u32(&sm->empty[group]), phase ^ 1u, abort)) ok = false;
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                __syncwarp();
                if (lane == 0) {
                    if (rank == 0) mbar_arrive(smem_u32(&sm->full[group]));
                    else mbar_arrive_cluster(smem_u32(&sm->full[group]), 0);
                }
                seq0 += P_STAGES;
                continue;
            }
            pair_group_bar(group);
            for (int q = 0; q < 2; ++q) {
                const long long rt = nt * 2 + (q == 0 ? rank : 1 - rank);
                for (int ks = tid; ks <= n_stages; ks += P_DEC_THREADS) {
                    uint4 v = __ldg(reinterpret_cast<const uint4 *>(&recs[rt * n_stages + ks]));
                    if (ks == n_stages) v.w = 0;
                    my_rec[q * (n_stages + 1) + ks] = v;
                }
            }
            pair_group_bar(group);
            if (gwarp == 0) {
                int n = 0;
                for (int k0 = 0; k0 < n_stages; k0 += 32) {
                    const int ks = k0 + lane;
                    unsigned l = 0;
                    if (ks < n_stages) l = my_rec[ks].w | my_rec[(n_stages + 1) + ks].w;
                    const unsigned m = __ballot_sync(0xffffffffu, l != 0);
                    if (l) my_list[n + __popc(m & ((1u << lane) - 1u))] = (unsigned short)ks;
                    n += __popc(m);
                }
                if (lane == 0) sm->n_live[group] = n;
            }
            pair_group_bar(group);
            const int n_live = sm->n_live[group];
            prev_nt = nt;
            prev_live = n_live;
            int i = (int)((group + P_GROUPS - (seq0 % P_GROUPS)) % P_GROUPS);
            if (i < n_live) { rec_at(my_list[i], &fr0, &fr1); fetch_entries<BW, P_DEC_THREADS>(fr0, fr1, p, tid, m0, m1); }
            for (; i < n_live; i += P_GROUPS) {
                const long long my_seq = seq0 + i;
                const int stage = group;
                const unsigned phase = (unsigned)((my_seq / P_STAGES) & 1);
                if (!mbar_wait(smem_u32(&sm->empty[stage]), phase ^ 1u, abort)) ok = false;
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                write_entries<BW, P_DEC_THREADS>(sB + stage * P_B_BYTES, fr0, fr1, p, tid, m0, m1);
                if (i + P_GROUPS < n_live) {
                    rec_at(my_list[i + P_GROUPS], &fr0, &fr1);
                    fetch_entries<BW, P_DEC_THREADS>(fr0, fr1, p, tid, m0, m1);
                }
                asm volatile("cp.async.wait_all;" ::: "memory");
                fence_proxy_async();
                __syncwarp();
                if (lane == 0) {
                    if (rank == 0) mbar_arrive(smem_u32(&sm->full[stage]));
                    else mbar_arrive_cluster(smem_u32(&sm->full[stage]), 0);
                }
            }
            seq0 += n_live;
        }
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

static size_t pair_smem_bytes(long long n_stages) {
    return 1024 + (size_t)P_STAGES * (P_A_BYTES + P_B_BYTES) + ((sizeof(PairSmem) + 15) & ~(size_t)15) +
           (size_t)P_GROUPS * 2 * (n_stages + 1) * 16 + (size_t)NEPI_WARPS * 2048;
}

bool pair_eligible(const Params &p) {
    return p.M > 256 && p.n_rec_tiles >= 2 && (p.n_rec_tiles % 2) == 0 && p.N % 256 == 0 &&
           p.n_stages <= MAX_STAGES_K && pair_smem_bytes(p.n_stages) <= 227 * 1024;
}

template <int BW>
static cudaError_t launch_pair_bw(const CUtensorMap &tmap, const Params &p, int sm_count, cudaStream_t st) {
    auto kern = mwu_gemm_pair_kernel<BW>;
    const size_t smem = pair_smem_bytes(p.n_stages);
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    const long long n_tiles = p.n_rec_tiles / 2;
    const long long tiles = ((p.M + 511) / 512) * n_tiles;
    long long pairs = sm_count / 2;
    if (tiles < pairs) pairs = tiles;
    Params q = p;
    // resident weights: the whole reduction fits the slots and every pair can own one weight tile
    q.resident = 0;
    if (p.n_stages <= P_STAGES && n_tiles <= pairs && tiles >= 4 * pairs) {
        q.resident = 1;
        pairs = pairs / n_tiles * n_tiles;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(2 * pairs));
    cfg.blockDim = dim3(P_THREADS);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    count_launch();
    return cudaLaunchKernelEx(&cfg, kern, tmap, q);
}

cudaError_t launch_pair(int bw, const CUtensorMap &tmap, const Params &p, int sm_count, cudaStream_t st) {
    switch (bw) {
        case 2: return launch_pair_bw<2>(tmap, p, sm_count, st);
        case 4: return launch_pair_bw<4>(tmap, p, sm_count, st);
        case 8: return launch_pair_bw<8>(tmap, p, sm_count, st);
        default: return launch_pair_bw<16>(tmap, p, sm_count, st);
    }
}

}  // namespace gemm
}  // namespace mwu
