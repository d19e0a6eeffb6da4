// Device-side building blocks shared by the GEMM kernels: constants, the kernel parameter block,
// PTX wrappers (mbarrier, TMA, tcgen05), shared-memory descriptors and the decode of the packed
// class lists into the swizzled K-major tile the tensor cores read.
#pragma once

#include <cuda.h>

#include "mwu_common.cuh"

namespace mwu {
namespace gemm {

constexpr int BMH = 128;                // rows of X per MMA (one half of a tile)
constexpr int BK = kStageK;             // 64
constexpr int STAGES = 3;
constexpr int AH_BYTES = BMH * BK * 2;  // 16 KiB: one 128-row half of the activation stage
constexpr int REC_BYTES = kTileRows * BK * 2;
constexpr int NDEC_GROUPS = STAGES;     // one decode group per pipeline slot
constexpr int NEPI_WARPS = 8;
constexpr int FIRST_DEC_WARP = 2 + NEPI_WARPS;
constexpr int MAX_GATHER_WARPS = 8;
// warps per decode group: six for the GEMM, four for the convolution (whose gather warps also
// need room inside the 1024-thread limit)
__host__ __device__ constexpr int dec_warps(int mode) { return mode ? 4 : 6; }
__host__ __device__ constexpr int first_gather_warp(int mode) { return FIRST_DEC_WARP + dec_warps(mode) * NDEC_GROUPS; }
__host__ __device__ constexpr int gather_warps(int mode, int mt) { return mode ? 4 * mt : 0; }
__host__ __device__ constexpr int cta_threads(int mode, int mt) {
    return 32 * (first_gather_warp(mode) + gather_warps(mode, mt));
}
constexpr int MAX_STAGES_K = 256;       // cols <= 16384
constexpr long long WAIT_LIMIT_CYCLES = 4000000000ll;   // about two seconds

// cuTensorMapEncodeTiled, looked up through the runtime (no link against the driver library)
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

struct Params {
    const unsigned char *packed;
    size_t off_rec, off_ulist, off_dpos, off_dpay, off_ppos;
    unsigned n_unified, n_dense, n_plist;   // list lengths, to keep every index in bounds
    long long n_rec_tiles;              // 128-row tiles of W
    long long n_stages;                 // K / 64
    long long M, N, K;
    void *Y;
    long long ldy;
    int y_fp32;
    int resident;                       // pair kernel: a CTA pair keeps one weight tile (see mwu_gemm2.cu)
    int stage_epi;                      // single-CTA GEMM: 16 KB of shared memory is there for store_chunk_staged
    int y_tma;                          // two-operand GEMM: bf16 output leaves through TMA stores (a tensor map of Y exists)
    int bw;                             // block width the descriptor names (checked against the packed header)
    int all_live;                       // two-operand GEMM on a plain dense matrix: no packed record table to consult
    unsigned *dev_status;
    // convolution only
    const __nv_bfloat16 *X;
    int C, H, W, KH, KW, stride, pad, OH, OW, NIMG;
    // staged gather (0 rows: gather straight from global memory instead)
    int patch_rows, patch_pitch, patch_nch;   // input rows per tile, row pitch (elements), channels per stage
};

// The packed buffer's header against what the host derived from the descriptor.  Every thread of
// every CTA evaluates it at kernel entry (the same few cached words), so the whole grid takes the
// same decision; on a mismatch the caller raises MWU_DEV_BOUNDS and returns before touching anything.
__device__ __forceinline__ bool header_matches(const Params &p) {
    const unsigned long long *h = reinterpret_cast<const unsigned long long *>(p.packed);
    return __ldg(h) == kMagic && __ldg(h + 2) == (unsigned long long)p.N && __ldg(h + 3) == (unsigned long long)p.K &&
           __ldg(h + 4) == (unsigned long long)p.bw && __ldg(h + 9) == (unsigned long long)p.n_unified &&
           __ldg(h + 10) == (unsigned long long)p.n_dense && __ldg(h + 11) == (unsigned long long)p.n_plist;
}
#define MWU_CHECK_HEADER(p)                                                        \
    do {                                                                           \
        if (!header_matches(p)) {                                                  \
            if (threadIdx.x == 0) atomicOr((p).dev_status, (unsigned)MWU_DEV_BOUNDS); \
            return;                                                                \
        }                                                                          \
    } while (0)

// ------------------------------------------------------------------------------------------
// PTX wrappers
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ unsigned smem_u32(const void *p) {
    return (unsigned)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(unsigned bar, unsigned count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(unsigned bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(unsigned bar, unsigned bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(unsigned bar, unsigned parity) {
    unsigned ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// non-blocking probe of a phase
__device__ __forceinline__ bool mbar_test(unsigned bar, unsigned parity) {
    unsigned ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// bounded wait: false when aborted or out of time (then *abort is set)
__device__ __forceinline__ bool mbar_wait(unsigned bar, unsigned parity, volatile int *abort) {
    // A short wait is polled (a waiter suspended in try_wait wakes a few hundred cycles late); a long
    // one, an epilogue warp waiting out a tile of a long reduction, sleeps in try_wait and leaves the
    // issue slots and the power to the warps that work.
#pragma unroll 1
    for (int i = 0; i < 128; ++i)
        if (mbar_test(bar, parity)) return true;
    const long long t0 = clock64();
#pragma unroll 1
    while (true) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*abort) return false;
        if (clock64() - t0 > WAIT_LIMIT_CYCLES) { *abort = 1; return false; }
    }
}
// the same for a single latency-critical warp (producer, MMA issuer): polled for much longer first
__device__ __forceinline__ bool mbar_wait_spin(unsigned bar, unsigned parity, volatile int *abort) {
#pragma unroll 1
    for (int i = 0; i < 4096; ++i)
        if (mbar_test(bar, parity)) return true;
    return mbar_wait(bar, parity, abort);
}
template <int BYTES>
__device__ __forceinline__ void cp_async_if(unsigned dst, const void *src, unsigned pred) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.u32 p, %2, 0;\n\t"
        "@p cp.async.ca.shared.global [%0], [%1], %3;\n\t}"
        ::"r"(dst), "l"(src), "r"(pred), "n"(BYTES) : "memory");
}
// true in exactly one lane of a converged warp
__device__ __forceinline__ bool elect_one() {
    unsigned pred;
    asm volatile("{\n\t.reg .pred p;\n\telect.sync _|p, 0xffffffff;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(pred));
    return pred != 0;
}
__device__ __forceinline__ void fence_proxy_async() {
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tma_load_2d(unsigned dst, const CUtensorMap *map, unsigned bar, int x, int y) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void tmem_alloc(unsigned dst_smem, unsigned ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(ncols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(unsigned taddr, unsigned ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void umma_bf16(unsigned d_tmem, unsigned long long adesc, unsigned long long bdesc,
                                          unsigned idesc, unsigned accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(unsigned bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// ---- CTA pairs (clusters of two, tcgen05 cta_group::2) ----
__device__ __forceinline__ unsigned cluster_rank() {
    unsigned r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// arrive on the barrier at the same shared-memory offset in CTA `cta` of the cluster
__device__ __forceinline__ void mbar_arrive_cluster(unsigned local_bar, unsigned cta) {
    unsigned remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_bar), "r"(cta));
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(remote) : "memory");
}
// address of the barrier at the same shared-memory offset in CTA `cta` of the cluster
__device__ __forceinline__ unsigned mbar_addr_in_cta(unsigned local_bar, unsigned cta) {
    unsigned remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_bar), "r"(cta));
    return remote;
}
// TMA load of a CTA pair: the data lands in this CTA's shared memory, the bytes are reported to a
// barrier that may live in either CTA of the pair (`bar_cluster` is a shared::cluster address).
// No multicast: each CTA fetches its own box.
__device__ __forceinline__ void tma_load_2d_pair(unsigned dst, const CUtensorMap *map, unsigned bar_cluster,
                                                 int x, int y) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.cta_group::2 "
        "[%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar_cluster), "r"(x), "r"(y) : "memory");
}
// shared memory -> global tile store; the box is clipped at the tensor's bounds
__device__ __forceinline__ void tma_store_2d(const CUtensorMap *map, unsigned src, int x, int y) {
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
                 ::"l"(map), "r"(src), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// the issuing thread's earlier bulk stores have read their shared-memory source
__device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
// ... all but the latest one have
__device__ __forceinline__ void bulk_wait_read_1() { asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory"); }
// ... and have completed
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

__device__ __forceinline__ void tmem_alloc2(unsigned dst_smem, unsigned ncols) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(ncols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc2(unsigned taddr, unsigned ncols) {
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void umma2_bf16(unsigned d_tmem, unsigned long long adesc, unsigned long long bdesc,
                                           unsigned idesc, unsigned accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// completion of all MMAs issued so far arrives on the barrier at this offset in both CTAs
__device__ __forceinline__ void umma2_commit_both(unsigned bar) {
    asm volatile(
        "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
        ::"r"(bar), "h"((unsigned short)3) : "memory");
}
// ... on the issuing CTA's barrier only
__device__ __forceinline__ void umma2_commit_local(unsigned bar) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// bf16 x bf16 -> fp32, both operands K-major, M = 256 over the CTA pair
__device__ __forceinline__ unsigned make_idesc_pair(int n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((unsigned)(n >> 3) << 17) | ((unsigned)(256 >> 4) << 24);
}

// issue a 32-lane x 32-column load from tensor memory; the registers are valid after tmem_ld_wait
__device__ __forceinline__ void tmem_ld32_issue(unsigned taddr, unsigned (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
}
// wait for all tensor-memory loads of this thread; the registers are passed through so that the
// compiler orders every later use of them after the wait
__device__ __forceinline__ void tmem_ld_wait(unsigned (&r)[32]) {
    asm volatile(
        "tcgen05.wait::ld.sync.aligned;"
        : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]),
          "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15]),
          "+r"(r[16]), "+r"(r[17]), "+r"(r[18]), "+r"(r[19]), "+r"(r[20]), "+r"(r[21]), "+r"(r[22]), "+r"(r[23]),
          "+r"(r[24]), "+r"(r[25]), "+r"(r[26]), "+r"(r[27]), "+r"(r[28]), "+r"(r[29]), "+r"(r[30]), "+r"(r[31])
        :: "memory");
}
__device__ __forceinline__ void tmem_ld32(unsigned taddr, unsigned (&r)[32]) {
    tmem_ld32_issue(taddr, r);
    tmem_ld_wait(r);
}

// a chunk of NC (16 or 32) columns of an output row: fp32 accumulators -> bf16 or fp32 -> global
template <int NC>
__device__ __forceinline__ void store_row_chunk(const Params &p, long long m, long long n0, const unsigned (&v)[NC]) {
    if (m >= p.M) return;
    if (p.y_fp32) {
        float *dst = reinterpret_cast<float *>(p.Y) + m * p.ldy + n0;
        if (n0 + NC <= p.N) {
#pragma unroll
            for (int j = 0; j < NC; j += 4)
                *reinterpret_cast<uint4 *>(dst + j) = make_uint4(v[j], v[j + 1], v[j + 2], v[j + 3]);
        } else {
            for (int j = 0; j < NC; ++j)
                if (n0 + j < p.N) dst[j] = __uint_as_float(v[j]);
        }
    } else {
        __nv_bfloat16 *dst = reinterpret_cast<__nv_bfloat16 *>(p.Y) + m * p.ldy + n0;
        if (n0 + NC <= p.N) {
#pragma unroll
            for (int j = 0; j < NC; j += 8) {
                uint4 o;
                __nv_bfloat162 h2;
                h2 = __floats2bfloat162_rn(__uint_as_float(v[j]), __uint_as_float(v[j + 1]));
                o.x = *reinterpret_cast<unsigned *>(&h2);
                h2 = __floats2bfloat162_rn(__uint_as_float(v[j + 2]), __uint_as_float(v[j + 3]));
                o.y = *reinterpret_cast<unsigned *>(&h2);
                h2 = __floats2bfloat162_rn(__uint_as_float(v[j + 4]), __uint_as_float(v[j + 5]));
                o.z = *reinterpret_cast<unsigned *>(&h2);
                h2 = __floats2bfloat162_rn(__uint_as_float(v[j + 6]), __uint_as_float(v[j + 7]));
                o.w = *reinterpret_cast<unsigned *>(&h2);
                *reinterpret_cast<uint4 *>(dst + j) = o;
            }
        } else {
            for (int j = 0; j < NC; ++j)
                if (n0 + j < p.N) dst[j] = __float2bfloat16_rn(__uint_as_float(v[j]));
        }
    }
}

// A 32-row x 32-column chunk of bf16 output, transposed through a 2 KB per-warp buffer so that four
// lanes write one 64-byte run of a row (whole 32-byte sectors) instead of 32 lanes writing 16 bytes
// to 32 different rows.  Lane l holds row mrow0 + l in v[]; row r keeps its four 16-byte pieces at
// positions j ^ ((r >> 1) & 3), which makes both the writes and the transposed reads conflict-free.
// All 32 lanes must call it; the caller guarantees n0 + 32 <= N and 16-byte aligned rows.
__device__ __forceinline__ void store_chunk_staged(const Params &p, long long mrow0, int lane, long long n0,
                                                   const unsigned (&v)[32], unsigned char *stg) {
    __syncwarp();
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        uint4 o;
        __nv_bfloat162 h2;
        h2 = __floats2bfloat162_rn(__uint_as_float(v[8 * j]), __uint_as_float(v[8 * j + 1]));
        o.x = *reinterpret_cast<unsigned *>(&h2);
        h2 = __floats2bfloat162_rn(__uint_as_float(v[8 * j + 2]), __uint_as_float(v[8 * j + 3]));
        o.y = *reinterpret_cast<unsigned *>(&h2);
        h2 = __floats2bfloat162_rn(__uint_as_float(v[8 * j + 4]), __uint_as_float(v[8 * j + 5]));
        o.z = *reinterpret_cast<unsigned *>(&h2);
        h2 = __floats2bfloat162_rn(__uint_as_float(v[8 * j + 6]), __uint_as_float(v[8 * j + 7]));
        o.w = *reinterpret_cast<unsigned *>(&h2);
        *reinterpret_cast<uint4 *>(stg + lane * 64 + ((j ^ ((lane >> 1) & 3)) << 4)) = o;
    }
    __syncwarp();
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int r = (lane >> 2) + 8 * i, pc = lane & 3;
        const uint4 o = *reinterpret_cast<const uint4 *>(stg + r * 64 + ((pc ^ ((r >> 1) & 3)) << 4));
        if (mrow0 + r < p.M)
            *reinterpret_cast<uint4 *>(reinterpret_cast<__nv_bfloat16 *>(p.Y) + (mrow0 + r) * p.ldy + n0 + pc * 8) = o;
    }
}

// K-major operand, 128-byte swizzle: rows of 128 bytes, 8-row groups 1024 bytes apart
__device__ __forceinline__ unsigned long long make_desc(unsigned smem_addr) {
    unsigned long long d = 0;
    d |= (unsigned long long)((smem_addr & 0x3FFFFu) >> 4);
    d |= (unsigned long long)1 << 16;                    // leading byte offset (unused for this layout)
    d |= (unsigned long long)(1024 >> 4) << 32;          // stride between 8-row groups
    d |= (unsigned long long)1 << 46;                    // descriptor version of this architecture
    d |= (unsigned long long)2 << 61;                    // 128-byte swizzle
    return d;
}
// bf16 x bf16 -> fp32, both operands K-major, M = 128
__device__ __forceinline__ unsigned make_idesc(int n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((unsigned)(n >> 3) << 17) | ((unsigned)(BMH >> 4) << 24);
}

// byte offset of 16-byte chunk c of row r inside a swizzled K-major tile
__device__ __forceinline__ unsigned swz(unsigned r, unsigned c) {
    return (r >> 3) * 1024u + (r & 7u) * 128u + ((c ^ (r & 7u)) << 4);
}

// ------------------------------------------------------------------------------------------
// decode of one record's class lists into its 128 x 64 tile
// ------------------------------------------------------------------------------------------
// One record = 128 * 64/BW block slots, listed as [pruned | dense | unified]; every entry names
// the byte offset of its block in the tile.  The three lists are laid end to end, each padded
// to a multiple of 8 entries, and thread `tid` of a decode group takes entries tid,
// tid+NDEC_THREADS, ... of that sequence, so the 8 lanes of a quarter warp always hold 8
// neighbouring entries of one list, which the packer ordered to fall into different banks.
// The work is split in two: fetch_entries reads the small per-entry words (it can run before the
// pipeline slot is free), write_entries fills the tile: zeros for pruned blocks, sign . bf16(u)
// for unified blocks, and an asynchronous global->shared copy of the stored values for dense ones.
template <int BW, int NDEC_THREADS>
struct DecodeCfg {
    static constexpr int NBK = BK / BW;
    static constexpr int SLOTS = kTileRows * NBK;
    static constexpr int ENT = (SLOTS + 24 + NDEC_THREADS - 1) / NDEC_THREADS;
    static constexpr int WORDS = BW / 2;                    // 32-bit words per block
    static constexpr unsigned OFF_MASK = (unsigned)(REC_BYTES - 1) & ~(unsigned)((BW >= 8 ? 16 : 2 * BW) - 1);
};

template <int BW, int NDEC_THREADS>
__device__ __forceinline__ void fetch_entries(const PackedRec r0, const PackedRec r1, const Params &p, int tid,
                                              unsigned (&m0)[DecodeCfg<BW, NDEC_THREADS>::ENT],
                                              unsigned (&m1)[DecodeCfg<BW, NDEC_THREADS>::ENT]) {
    constexpr int ENT = DecodeCfg<BW, NDEC_THREADS>::ENT;
    const uint2 *ulist = reinterpret_cast<const uint2 *>(p.packed + p.off_ulist);
    const unsigned short *dpos = reinterpret_cast<const unsigned short *>(p.packed + p.off_dpos);
    const unsigned short *ppos = reinterpret_cast<const unsigned short *>(p.packed + p.off_ppos);
    const unsigned n_p = r1.pbase - r0.pbase, n_d = r1.dbase - r0.dbase, n_u = r1.ubase - r0.ubase;
    const unsigned p8 = (n_p + 7u) & ~7u, d8 = (n_d + 7u) & ~7u;
#pragma unroll
    for (int k = 0; k < ENT; ++k) {
        const unsigned f = (unsigned)tid + (unsigned)k * NDEC_THREADS;
        m0[k] = 0xffffffffu;                                // nothing to write
        m1[k] = 0u;
        if (f < p8) {
            const unsigned e = r0.pbase + f;
            if (f < n_p && e < p.n_plist) m0[k] = __ldg(ppos + e);
        } else if (f < p8 + d8) {
            const unsigned e = r0.dbase + (f - p8);
            if (f - p8 < n_d && e < p.n_dense) m0[k] = __ldg(dpos + e);
        } else if (f - p8 - d8 < n_u) {
            const unsigned e = r0.ubase + (f - p8 - d8);
            if (e < p.n_unified) {
                const uint2 ent = __ldg(ulist + e);          // x: spread signs, y: off | bf16(u) << 16
                m0[k] = ent.y;
                m1[k] = ent.x;
            }
        }
    }
}

template <int BW, int NDEC_THREADS>
__device__ __forceinline__ void write_entries(unsigned char *tile, const PackedRec r0, const PackedRec r1,
                                              const Params &p, int tid,
                                              const unsigned (&m0)[DecodeCfg<BW, NDEC_THREADS>::ENT],
                                              const unsigned (&m1)[DecodeCfg<BW, NDEC_THREADS>::ENT]) {
    constexpr int ENT = DecodeCfg<BW, NDEC_THREADS>::ENT;
    constexpr int WORDS = DecodeCfg<BW, NDEC_THREADS>::WORDS;
    constexpr unsigned OFF_MASK = DecodeCfg<BW, NDEC_THREADS>::OFF_MASK;
    const unsigned char *dpay = p.packed + p.off_dpay;
    const unsigned n_p = r1.pbase - r0.pbase, n_d = r1.dbase - r0.dbase;
    const unsigned p8 = (n_p + 7u) & ~7u, d8 = (n_d + 7u) & ~7u;
    const unsigned tile_s = smem_u32(tile);
    // no branches per entry: every entry computes its words (zero unless unified), stores them
    // unless it is dense, and issues its copy if it is dense
#pragma unroll
    for (int k = 0; k < ENT; ++k) {
        const unsigned f = (unsigned)tid + (unsigned)k * NDEC_THREADS;
        const bool valid = m0[k] != 0xffffffffu;
        const unsigned off = m0[k] & OFF_MASK;
        const bool is_d = (f - p8) < d8;                    // unsigned: also false for f < p8
        const bool is_u = f >= p8 + d8;
        const unsigned umask = is_u ? 0xffffffffu : 0u;
        const unsigned u2 = __byte_perm(m0[k], 0u, 0x3232);  // bf16(u) in both halves
        unsigned w[8];
#pragma unroll
        for (int q = 0; q < 8; ++q)                          // weights 2q, 2q+1: sign bits q and 16+q
            w[q] = (q < WORDS) ? ((((m1[k] << (15 - q)) & 0x80008000u) ^ u2) & umask) : 0u;
        const unsigned char *src = dpay + (size_t)(r0.dbase + (f - p8)) * (2 * BW);
        const unsigned do_copy = (valid && is_d) ? 1u : 0u;
        const bool do_store = valid && !is_d;
        if (BW == 16) {
            cp_async_if<16>(tile_s + off, src, do_copy);
            cp_async_if<16>(tile_s + (off ^ 16u), src + 16, do_copy);
            if (do_store) {
                *reinterpret_cast<uint4 *>(tile + off) = make_uint4(w[0], w[1], w[2], w[3]);
                *reinterpret_cast<uint4 *>(tile + (off ^ 16u)) = make_uint4(w[4], w[5], w[6], w[7]);
            }
        } else if (BW == 8) {
            cp_async_if<16>(tile_s + off, src, do_copy);
            if (do_store) *reinterpret_cast<uint4 *>(tile + off) = make_uint4(w[0], w[1], w[2], w[3]);
        } else if (BW == 4) {
            cp_async_if<8>(tile_s + off, src, do_copy);
            if (do_store) *reinterpret_cast<uint2 *>(tile + off) = make_uint2(w[0], w[1]);
        } else {
            cp_async_if<4>(tile_s + off, src, do_copy);
            if (do_store) *reinterpret_cast<unsigned *>(tile + off) = w[0];
        }
    }
}

}  // namespace gemm
}  // namespace mwu
