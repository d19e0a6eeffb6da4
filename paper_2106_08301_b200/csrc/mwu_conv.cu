// mwu_conv_implicit_ws: the convolution as an implicit GEMM over weights expanded once per call.
//
// The fused kernel behind mwu_conv_implicit decodes every weight record again for each activation
// tile and assembles its im2col rows element by element.  With a workspace the work is split:
//   conv_prep_kernel        one launch, two jobs side by side: image tiles are copied into
//                           pixel-major order (channels innermost, so that the 64 channels of a
//                           pixel are one 128-byte line), and the packed weights are expanded once,
//                           as mwu_decode does, but with the reduction axis tap-major: column
//                           (i*kw + j) * cin + c instead of c * kh*kw + i*kw + j (the same products,
//                           summed tap by tap);
//   mwu_conv_taps_kernel    one CTA per tile of R output rows x OW pixels (R * OW <= 128) and 128
//                           filters.  A k stage is one filter tap and 64 channels: its activation
//                           operand is a box of the pixel-major image shifted by the tap's offset,
//                           fetched by ONE tiled TMA load whose out-of-range rows and columns read
//                           as zero (the padding costs nothing and no im2col row is ever built);
//                           its weight operand is a 128 x 64 box of the expanded weights.
//                           tcgen05.mma 128 x 128 x 16, fp32 accumulators double-buffered in
//                           tensor memory, so the epilogue of a tile runs under the next tile's loop.
// Roles (6 warps): warp 0 issues the TMA loads, warp 1 owns tensor memory and issues the MMAs,
// warps 2-5 read the accumulators and store NCHW output (a lane is a pixel, so the 32 lanes of a
// warp write 32 neighbouring pixels of one filter: one 64-byte run).
// Every wait on an mbarrier is bounded; when one runs out the kernel raises MWU_DEV_TIMEOUT, waits
// for the loads it has in flight, frees its tensor memory and returns.
#include "mwu_gemm_dev.cuh"

namespace mwu {
namespace gemm {

EncodeTiledFn get_encode_fn();          // mwu_gemm.cu

constexpr int C_STAGES = 6;
constexpr int C_A_BYTES = 128 * 128;    // up to 128 pixels x 64 channels
constexpr int C_B_BYTES = REC_BYTES;    // 128 filters x 64 channels
constexpr int C_THREADS = 32 * 6;

struct ConvParams {
    Params g;                           // packed weights, N = filters, K = cin*kh*kw, Y, y_fp32, dev_status
    int C, H, W, KH, KW, pad, OH, OW, NIMG;
    int R;                              // output rows per tile
    int tiles_per_img;
    int n_ntiles;                       // 128-filter tiles
    unsigned a_bytes;                   // bytes one activation load delivers
    long long wait_limit;               // cycles a wait may take
    long long withhold;                 // testing aid: running number of a stage whose loads are left out (-1: none)
};

struct ConvSmem {
    unsigned long long full[C_STAGES], empty[C_STAGES], tfull[2], tempty[2], drain;
    unsigned tmem_base;
    int abort;
};

__device__ __forceinline__ bool mbar_wait_lim(unsigned bar, unsigned parity, volatile int *abort, long long limit) {
    if (mbar_test(bar, parity)) return true;
#pragma unroll 1
    for (int i = 0; i < 128; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
#pragma unroll 1
    while (true) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*abort) return false;
        if (clock64() - t0 > limit) { *abort = 1; return false; }
    }
}

__device__ __forceinline__ void tma_load_4d(unsigned dst, const CUtensorMap *map, unsigned bar, int c0, int c1,
                                            int c2, int c3) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}

// ------------------------------------------------------------------------------------------
// preparation, one launch: the input image [n][c][h*w] -> [n][h*w][c], and the weights
// ------------------------------------------------------------------------------------------
constexpr int PREP_THREADS = 512;

// one CTA: a tile of 64 pixels x 64 channels of one image, read as pixel pairs, written as channel pairs
__device__ __forceinline__ void nchw_to_nhwc_tile(const unsigned short *x, unsigned short *xt, int C, int HW,
                                                  int tile, int tiles_hw, int tiles_c) {
    __shared__ unsigned short s_t[64][66];
    const int img = tile / (tiles_hw * tiles_c), rem = tile % (tiles_hw * tiles_c);
    const int hw0 = (rem % tiles_hw) * 64, c0 = (rem / tiles_hw) * 64;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;            // 32 x 16
    const long long base = (long long)img * C * HW;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int c = c0 + ty + 16 * i, hw = hw0 + 2 * tx;
        unsigned short a = 0, b = 0;
        if (c < C) {
            if (hw + 1 < HW && (HW & 1) == 0) {
                const unsigned v = *reinterpret_cast<const unsigned *>(x + base + (long long)c * HW + hw);
                a = (unsigned short)v; b = (unsigned short)(v >> 16);
            } else {
                if (hw < HW) a = x[base + (long long)c * HW + hw];
                if (hw + 1 < HW) b = x[base + (long long)c * HW + hw + 1];
            }
        }
        s_t[ty + 16 * i][2 * tx] = a;
        s_t[ty + 16 * i][2 * tx + 1] = b;
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int hw = hw0 + ty + 16 * i, c = c0 + 2 * tx;
        if (hw < HW && c + 1 < C + 1) {
            unsigned short *dst = xt + ((long long)img * HW + hw) * C + c;
            const unsigned short a = s_t[2 * tx][ty + 16 * i], b = s_t[2 * tx + 1][ty + 16 * i];
            if (c + 1 < C) *reinterpret_cast<unsigned *>(dst) = (unsigned)a | ((unsigned)b << 16);     // C is even
            else if (c < C) dst[0] = a;
        }
    }
}

// one CTA: a packed 128 x 64 record -> row-major bf16 with the reduction axis in tap-major order
template <int BW>
__device__ __forceinline__ void decode_taps_record(const Params &p, unsigned short *Wd, int taps, int C, long long rec) {
    __shared__ __align__(1024) unsigned char tile[REC_BYTES];
    constexpr int ENT = DecodeCfg<BW, PREP_THREADS>::ENT;
    const PackedRec *recs = reinterpret_cast<const PackedRec *>(p.packed + p.off_rec);
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
    fetch_entries<BW, PREP_THREADS>(r0, r1, p, tid, m0, m1);
    write_entries<BW, PREP_THREADS>(tile, r0, r1, p, tid, m0, m1);
    asm volatile("cp.async.wait_all;" ::: "memory");
    __syncthreads();
#pragma unroll
    for (int i = 0; i < (REC_BYTES / 16) / PREP_THREADS; ++i) {
        const int q = tid + i * PREP_THREADS;               // 16-byte piece: row q / 8, piece q % 8
        const int r = q >> 3, j = q & 7;
        const uint4 v = *reinterpret_cast<const uint4 *>(tile + r * 128 + ((j ^ (r & 7)) << 4));
        const unsigned wds[4] = {v.x, v.y, v.z, v.w};
        unsigned short *row = Wd + (rt * kTileRows + r) * p.K;
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const int k = (int)ks * BK + j * 8 + e;         // column in [c][tap] order
            const int c = k / taps, tap = k - c * taps;
            row[(long long)tap * C + c] = (unsigned short)(wds[e >> 1] >> (16 * (e & 1)));
        }
    }
}

// CTAs [0, n_rec): weight records; the rest: image tiles.  The two jobs do not depend on each other,
// so one launch runs them side by side.
template <int BW>
__global__ void __launch_bounds__(PREP_THREADS) conv_prep_kernel(const Params p, unsigned short *Wd, int taps, int C,
                                                                 unsigned n_rec, const unsigned short *x,
                                                                 unsigned short *xt, int HW, int tiles_hw, int tiles_c) {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the tensor-core kernel may set itself up meanwhile
    if (blockIdx.x < n_rec) {
        MWU_CHECK_HEADER(p);
        decode_taps_record<BW>(p, Wd, taps, C, blockIdx.x);
    } else {
        nchw_to_nhwc_tile(x, xt, C, HW, (int)(blockIdx.x - n_rec), tiles_hw, tiles_c);
    }
}

// the image alone (weights come from somewhere else)
__global__ void __launch_bounds__(PREP_THREADS) nchw_to_nhwc_kernel(const unsigned short *x, unsigned short *xt, int C,
                                                                    int HW, int tiles_hw, int tiles_c) {
    nchw_to_nhwc_tile(x, xt, C, HW, (int)blockIdx.x, tiles_hw, tiles_c);
}

// a plain dense weight matrix [rows][ldw] in [c][tap] column order -> [n_pad][c * taps] tap-major
// (rows beyond `rows` are written as zeros)
__global__ void __launch_bounds__(256) permute_taps_kernel(const unsigned short *Wd, long long ldw, long long rows,
                                                           long long n_pad, int taps, int C, unsigned short *out) {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const long long K = (long long)taps * C, total = n_pad * K;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
        const long long row = i / K, kk = i - row * K;
        const int tap = (int)(kk / C), c = (int)(kk - (long long)tap * C);
        out[i] = row < rows ? Wd[row * ldw + (long long)c * taps + tap] : (unsigned short)0;
    }
}

// ------------------------------------------------------------------------------------------
// the tensor-core kernel
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(C_THREADS, 1)
mwu_conv_taps_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_w,
                     const ConvParams p) {
    if (!p.g.all_live) MWU_CHECK_HEADER(p.g);
    extern __shared__ unsigned char smem_raw[];
    unsigned char *base = reinterpret_cast<unsigned char *>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    unsigned char *sA = base;
    unsigned char *sB = base + C_STAGES * C_A_BYTES;
    ConvSmem *sm = reinterpret_cast<ConvSmem *>(sB + C_STAGES * C_B_BYTES);
    volatile int *abort = &sm->abort;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int chunks = p.C / BK;                            // 64-channel chunks
    const int n_ks = p.KH * p.KW * chunks;                  // k stages per tile
    const long long total_tiles = (long long)p.NIMG * p.tiles_per_img * p.n_ntiles;
    const long long limit = p.wait_limit;

    if (threadIdx.x == 0) {
        for (int s = 0; s < C_STAGES; ++s) {
            mbar_init(smem_u32(&sm->full[s]), 1);
            mbar_init(smem_u32(&sm->empty[s]), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&sm->tfull[b]), 1);
            mbar_init(smem_u32(&sm->tempty[b]), 4);
        }
        mbar_init(smem_u32(&sm->drain), 1);
        sm->abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(smem_u32(&sm->tmem_base), 256);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    // launched with programmatic stream serialization: the set-up above ran while the kernel that
    // prepares the operands was still finishing; its memory is complete from here on
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const unsigned tmem_base = *reinterpret_cast<volatile unsigned *>(&sm->tmem_base);

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        int stage = 0;
        unsigned phase = 0;
        bool ok = true;
        long long seq = 0;                                  // stages issued so far
        unsigned issued = 0, last_phase = 0;                // per slot: a load was issued; parity of its phase
        for (long long t = blockIdx.x; ok && t < total_tiles; t += gridDim.x) {
            const long long nt = t % p.n_ntiles, mt = t / p.n_ntiles;
            const int img = (int)(mt / p.tiles_per_img), oh0 = (int)(mt % p.tiles_per_img) * p.R;
            for (int ks = 0; ks < n_ks; ++ks) {
                if (!mbar_wait_lim(smem_u32(&sm->empty[stage]), phase ^ 1u, abort, limit)) ok = false;
                if (!__all_sync(0xffffffffu, ok)) { ok = false; break; }
                if (seq != p.withhold && elect_one()) {
                    const int tap = ks / chunks, cc = ks - tap * chunks;
                    const int di = tap / p.KW, dj = tap - di * p.KW;
                    const unsigned bar = smem_u32(&sm->full[stage]);
                    mbar_expect_tx(bar, p.a_bytes + C_B_BYTES);
                    tma_load_4d(smem_u32(sA + stage * C_A_BYTES), &tmap_x, bar, cc * BK, dj - p.pad, oh0 + di - p.pad, img);
                    tma_load_2d(smem_u32(sB + stage * C_B_BYTES), &tmap_w, bar, ks * BK, (int)(nt * kTileRows));
                }
                __syncwarp();
                if (seq != p.withhold) {
                    issued |= 1u << stage;
                    last_phase = (last_phase & ~(1u << stage)) | (phase << stage);
                }
                ++seq;
                if (++stage == C_STAGES) { stage = 0; phase ^= 1u; }
            }
        }
        if (!ok) {
            // leaving early: the loads already issued must have landed before the CTA goes away.  Their
            // barriers need nothing but the loads' own bytes, so these waits end (and are bounded anyway).
            __shared__ int s_no_abort;
            if (lane == 0) s_no_abort = 0;
            __syncwarp();
            for (int s = 0; s < C_STAGES; ++s)
                if ((issued >> s) & 1u) mbar_wait_lim(smem_u32(&sm->full[s]), (last_phase >> s) & 1u, &s_no_abort, limit);
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        int stage = 0;
        unsigned phase = 0;
        bool ok = true, issued_any = false;
        const unsigned idesc = make_idesc(128);
        long long k = 0;
        for (long long t = blockIdx.x; ok && t < total_tiles; t += gridDim.x, ++k) {
            const unsigned buf = (unsigned)(k & 1), use_phase = (unsigned)((k >> 1) & 1);
            if (!mbar_wait_lim(smem_u32(&sm->tempty[buf]), use_phase ^ 1u, abort, limit)) ok = false;
            if (!__all_sync(0xffffffffu, ok)) { ok = false; break; }
            tc_fence_after();
            for (int ks = 0; ks < n_ks; ++ks) {
                if (!mbar_wait_lim(smem_u32(&sm->full[stage]), phase, abort, limit)) ok = false;
                if (!__all_sync(0xffffffffu, ok)) { ok = false; break; }
                tc_fence_after();
                const unsigned long long adesc = make_desc(smem_u32(sA + stage * C_A_BYTES));
                const unsigned long long bdesc = make_desc(smem_u32(sB + stage * C_B_BYTES));
                if (elect_one()) {
#pragma unroll
                    for (int k4 = 0; k4 < 4; ++k4)
                        umma_bf16(tmem_base + buf * 128u, adesc + (unsigned long long)(k4 * 2),
                                  bdesc + (unsigned long long)(k4 * 2), idesc, (ks | k4) ? 1u : 0u);
                    umma_commit(smem_u32(&sm->empty[stage]));
                }
                issued_any = true;
                __syncwarp();
                if (++stage == C_STAGES) { stage = 0; phase ^= 1u; }
            }
            if (!ok) break;
            if (elect_one()) umma_commit(smem_u32(&sm->tfull[buf]));
            __syncwarp();
        }
        // everything this warp issued must have retired before tensor memory is freed
        if (lane == 0 && issued_any) {
            __shared__ int s_no_abort2;
            s_no_abort2 = 0;
            umma_commit(smem_u32(&sm->drain));
            mbar_wait_lim(smem_u32(&sm->drain), 0, &s_no_abort2, limit);
        }
        __syncwarp();
    } else {
        // ---------------- epilogue: TMEM lanes are pixels, columns are filters ----------------
        const int quarter = warp & 3;
        const int m = quarter * 32 + lane;                  // pixel of the tile
        bool ok = true;
        long long k = 0;
        const long long plane = (long long)p.OH * p.OW;
        for (long long t = blockIdx.x; ok && t < total_tiles; t += gridDim.x, ++k) {
            const long long nt = t % p.n_ntiles, mt = t / p.n_ntiles;
            const long long img = mt / p.tiles_per_img;
            const int oh0 = (int)(mt % p.tiles_per_img) * p.R;
            const unsigned buf = (unsigned)(k & 1), use_phase = (unsigned)((k >> 1) & 1);
            if (!mbar_wait_lim(smem_u32(&sm->tfull[buf]), use_phase, abort, limit)) ok = false;
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            const int rows_here = (p.OH - oh0) < p.R ? (p.OH - oh0) : p.R;
            const bool px_ok = m < rows_here * p.OW;
            const unsigned trow = tmem_base + ((unsigned)(quarter * 32) << 16) + buf * 128u;
            const long long pix = (long long)oh0 * p.OW + m;
#pragma unroll 1
            for (int c0 = 0; c0 < 128; c0 += 32) {
                const long long o0 = nt * kTileRows + c0;
                if (o0 >= p.g.N) break;
                unsigned v[32];
                tmem_ld32(trow + (unsigned)c0, v);
                if (px_ok) {
                    if (p.g.y_fp32) {
                        float *dst = reinterpret_cast<float *>(p.g.Y) + (img * p.g.N + o0) * plane + pix;
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (o0 + j < p.g.N) dst[j * plane] = __uint_as_float(v[j]);
                    } else {
                        __nv_bfloat16 *dst = reinterpret_cast<__nv_bfloat16 *>(p.g.Y) + (img * p.g.N + o0) * plane + pix;
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (o0 + j < p.g.N) dst[j * plane] = __float2bfloat16_rn(__uint_as_float(v[j]));
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sm->tempty[buf]));
        }
    }

    // teardown
    tc_fence_before();
    __syncthreads();
    // after the barrier: a role that finished its own work early must still see a flag raised later
    if (*abort && threadIdx.x == 0) atomicOr(p.g.dev_status, (unsigned)MWU_DEV_TIMEOUT);
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 256);
    }
}

static size_t conv_smem_bytes() { return 1024 + (size_t)C_STAGES * (C_A_BYTES + C_B_BYTES) + sizeof(ConvSmem); }

// shape served by the workspace path?  Fills the tile geometry when it is.
static bool taps_path(const mwu_proj_desc *desc, int n, int c, int h, int w, int kh, int kw, int stride, int pad,
                      int *OH, int *OW, int *R) {
    if (validate_desc(desc, true) != MWU_OK) return false;
    if (n <= 0 || c <= 0 || h <= 0 || w <= 0 || kh <= 0 || kw <= 0 || stride != 1 || pad < 0) return false;
    if ((int64_t)c * kh * kw != desc->cols || c % BK != 0) return false;
    if (h + 2 * pad < kh || w + 2 * pad < kw || pad > 32767) return false;
    const int oh = h + 2 * pad - kh + 1, ow = w + 2 * pad - kw + 1;
    if (ow > 128 || w > 65535 || h > 65535) return false;
    int r = 128 / ow;
    if (r > oh) r = oh;
    if (r > 256) r = 256;
    *OH = oh; *OW = ow; *R = r;
    return true;
}

static size_t x_bytes_aligned(int n, int c, int h, int w) { return align_up((size_t)n * c * h * w * 2, 1024); }

// testing aid (see mwu.h): limit of the bounded waits and a stage to leave out
static long long g_wait_limit = WAIT_LIMIT_CYCLES;
static long long g_withhold = -1;

}  // namespace gemm
}  // namespace mwu

extern "C" void mwu_debug_conv_wait(int64_t limit_cycles, int64_t withhold_stage) {
    mwu::gemm::g_wait_limit = limit_cycles > 0 ? limit_cycles : mwu::gemm::WAIT_LIMIT_CYCLES;
    mwu::gemm::g_withhold = withhold_stage;
}

extern "C" size_t mwu_conv_workspace_bytes(const mwu_proj_desc *desc, int32_t n, int32_t c, int32_t h,
                                           int32_t w, int32_t kh, int32_t kw, int32_t stride, int32_t pad) {
    using namespace mwu;
    int OH, OW, R;
    if (!gemm::taps_path(desc, n, c, h, w, kh, kw, stride, pad, &OH, &OW, &R)) return 0;
    const PackedLayout L = packed_layout(desc);
    return gemm::x_bytes_aligned(n, c, h, w) + (size_t)L.n_pad * (size_t)desc->cols * 2;
}

namespace mwu {
namespace gemm {

// shape of the convolution alone (no descriptor): stride 1, channels in chunks of 64, at most 128
// output pixels per row
static bool taps_geometry(int n, int c, int h, int w, int kh, int kw, int stride, int pad, int *OH, int *OW, int *R) {
    if (n <= 0 || c <= 0 || h <= 0 || w <= 0 || kh <= 0 || kw <= 0 || stride != 1 || pad < 0) return false;
    if (c % BK != 0 || h + 2 * pad < kh || w + 2 * pad < kw || pad > 32767) return false;
    const int oh = h + 2 * pad - kh + 1, ow = w + 2 * pad - kw + 1;
    if (ow > 128 || w > 65535 || h > 65535) return false;
    int r = 128 / ow;
    if (r > oh) r = oh;
    if (r > 256) r = 256;
    *OH = oh; *OW = ow; *R = r;
    return true;
}

// tensor maps, the preparation (`prepare` enqueues the image copy and whatever puts the tap-major
// weights into `wd`) and the tensor-core kernel
template <typename F>
static int run_taps(ConvParams &p, const void *X_nchw, int n, int c, int h, int w, int kh, int kw, int pad,
                    unsigned short *xt, unsigned short *wd, long long n_pad, int sm_count, cudaStream_t st,
                    F prepare) {
    EncodeTiledFn encode = get_encode_fn();
    if (!encode) return MWU_ERR_CUDA;
    int OH, OW, R;
    if (!taps_geometry(n, c, h, w, kh, kw, 1, pad, &OH, &OW, &R)) return MWU_ERR_SHAPE;
    const long long K = (long long)c * kh * kw;
    p.C = c; p.H = h; p.W = w; p.KH = kh; p.KW = kw; p.pad = pad; p.OH = OH; p.OW = OW; p.NIMG = n;
    p.R = R;
    p.tiles_per_img = (OH + R - 1) / R;
    p.n_ntiles = (int)(n_pad / kTileRows);
    p.a_bytes = (unsigned)(R * OW * 128);
    p.wait_limit = g_wait_limit;
    p.withhold = g_withhold;
    // tensor maps: the pixel-major image as [n][h][w][c] (innermost first: c, w, h, n), and the weights
    CUtensorMap tmap_x, tmap_w;
    {
        const cuuint64_t gdim[4] = {(cuuint64_t)c, (cuuint64_t)w, (cuuint64_t)h, (cuuint64_t)n};
        const cuuint64_t gstr[3] = {(cuuint64_t)c * 2, (cuuint64_t)w * c * 2, (cuuint64_t)h * w * c * 2};
        const cuuint32_t box[4] = {(cuuint32_t)BK, (cuuint32_t)OW, (cuuint32_t)R, 1};
        const cuuint32_t estr[4] = {1, 1, 1, 1};
        if (encode(&tmap_x, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, xt, gdim, gstr, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                   CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return MWU_ERR_CUDA;
        const cuuint64_t wdim[2] = {(cuuint64_t)K, (cuuint64_t)n_pad};
        const cuuint64_t wstr[1] = {(cuuint64_t)K * 2};
        const cuuint32_t wbox[2] = {(cuuint32_t)BK, (cuuint32_t)kTileRows};
        const cuuint32_t west[2] = {1, 1};
        if (encode(&tmap_w, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, wd, wdim, wstr, wbox, west, CU_TENSOR_MAP_INTERLEAVE_NONE,
                   CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return MWU_ERR_CUDA;
    }
    const int HW = h * w;
    const int tiles_hw = (HW + 63) / 64, tiles_c = (c + 63) / 64;
    prepare((const unsigned short *)X_nchw, xt, HW, tiles_hw, tiles_c, (unsigned)(n * tiles_hw * tiles_c));
    const size_t smem = conv_smem_bytes();
    if (cudaFuncSetAttribute(mwu_conv_taps_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return MWU_ERR_CUDA;
    const long long tiles = (long long)n * p.tiles_per_img * p.n_ntiles;
    const int grid = (int)(tiles < sm_count ? tiles : sm_count);
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(C_THREADS);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    count_launch();
    if (cudaLaunchKernelEx(&cfg, mwu_conv_taps_kernel, tmap_x, tmap_w, p) != cudaSuccess) return MWU_ERR_CUDA;
    return cudaGetLastError() == cudaSuccess ? MWU_OK : MWU_ERR_CUDA;
}

}  // namespace gemm
}  // namespace mwu

extern "C" int mwu_conv_implicit_ws(const mwu_proj_desc *desc, const void *packed, const void *X_nchw,
                                    int32_t n, int32_t c, int32_t h, int32_t w, int32_t kh, int32_t kw,
                                    int32_t stride, int32_t pad, void *Y_nchw, int32_t y_dtype,
                                    void *workspace, size_t workspace_bytes, uint32_t *dev_status,
                                    void *cuda_stream) {
    using namespace mwu;
    using namespace mwu::gemm;
    const size_t need = mwu_conv_workspace_bytes(desc, n, c, h, w, kh, kw, stride, pad);
    if (!workspace || need == 0 || workspace_bytes < need)
        return mwu_conv_implicit(desc, packed, X_nchw, n, c, h, w, kh, kw, stride, pad, Y_nchw, y_dtype,
                                 dev_status, cuda_stream);
    if (!packed || !X_nchw || !Y_nchw || !dev_status) return MWU_ERR_INVALID_ARG;
    if (y_dtype != 0 && y_dtype != 1) return MWU_ERR_INVALID_ARG;
    if (!aligned_to(packed, 256) || !aligned_to(X_nchw, 16) || !aligned_to(Y_nchw, 16) ||
        !aligned_to(dev_status, 4) || !aligned_to(workspace, 256))
        return MWU_ERR_ALIGNMENT;
    int sm_count = 0;
    int rc = check_device(&sm_count);
    if (rc != MWU_OK) return rc;
    cudaStream_t st = (cudaStream_t)cuda_stream;

    ConvParams p = {};
    const PackedLayout L = packed_layout(desc);
    p.g.packed = (const unsigned char *)packed;
    p.g.off_rec = L.off_rec; p.g.off_ulist = L.off_ulist; p.g.off_dpos = L.off_dpos;
    p.g.off_dpay = L.off_dpay; p.g.off_ppos = L.off_ppos;
    p.g.n_unified = (unsigned)L.n_unified; p.g.n_dense = (unsigned)L.n_dense; p.g.n_plist = (unsigned)L.n_plist;
    p.g.n_rec_tiles = L.n_tiles;
    p.g.n_stages = L.n_stages;
    p.g.N = desc->rows;
    p.g.K = desc->cols;
    p.g.bw = desc->block;
    p.g.Y = Y_nchw;
    p.g.y_fp32 = y_dtype;
    p.g.dev_status = dev_status;
    unsigned short *xt = (unsigned short *)workspace;
    unsigned short *wd = (unsigned short *)((char *)workspace + x_bytes_aligned(n, c, h, w));
    const unsigned n_rec = (unsigned)(L.n_tiles * L.n_stages);
    const int taps = kh * kw, bw = desc->block;
    const Params g = p.g;
    return run_taps(p, X_nchw, n, c, h, w, kh, kw, pad, xt, wd, L.n_pad, sm_count, st,
                    [&](const unsigned short *x, unsigned short *xo, int HW, int tiles_hw, int tiles_c, unsigned n_tiles) {
        const unsigned grid = n_rec + n_tiles;
        switch (bw) {
            case 2: conv_prep_kernel<2><<<grid, PREP_THREADS, 0, st>>>(g, wd, taps, c, n_rec, x, xo, HW, tiles_hw, tiles_c); break;
            case 4: conv_prep_kernel<4><<<grid, PREP_THREADS, 0, st>>>(g, wd, taps, c, n_rec, x, xo, HW, tiles_hw, tiles_c); break;
            case 8: conv_prep_kernel<8><<<grid, PREP_THREADS, 0, st>>>(g, wd, taps, c, n_rec, x, xo, HW, tiles_hw, tiles_c); break;
            default: conv_prep_kernel<16><<<grid, PREP_THREADS, 0, st>>>(g, wd, taps, c, n_rec, x, xo, HW, tiles_hw, tiles_c); break;
        }
        count_launch();
    });
}

extern "C" size_t mwu_conv_dense_workspace_bytes(int64_t rows, int32_t n, int32_t c, int32_t h, int32_t w,
                                                 int32_t kh, int32_t kw, int32_t stride, int32_t pad) {
    using namespace mwu;
    int OH, OW, R;
    if (rows <= 0 || !gemm::taps_geometry(n, c, h, w, kh, kw, stride, pad, &OH, &OW, &R)) return 0;
    const int64_t n_pad = (rows + kTileRows - 1) / kTileRows * kTileRows;
    return gemm::x_bytes_aligned(n, c, h, w) + (size_t)n_pad * (size_t)c * kh * kw * 2;
}

extern "C" int mwu_conv_dense(int64_t rows, const void *Wd, int64_t ldw, const void *X_nchw, int32_t n, int32_t c,
                              int32_t h, int32_t w, int32_t kh, int32_t kw, int32_t stride, int32_t pad,
                              void *Y_nchw, int32_t y_dtype, void *workspace, size_t workspace_bytes,
                              uint32_t *dev_status, void *cuda_stream) {
    using namespace mwu;
    using namespace mwu::gemm;
    if (!Wd || !X_nchw || !Y_nchw || !dev_status || !workspace) return MWU_ERR_INVALID_ARG;
    if (y_dtype != 0 && y_dtype != 1) return MWU_ERR_INVALID_ARG;
    const size_t need = mwu_conv_dense_workspace_bytes(rows, n, c, h, w, kh, kw, stride, pad);
    if (need == 0 || ldw < (int64_t)c * kh * kw) return MWU_ERR_SHAPE;
    if (workspace_bytes < need) return MWU_ERR_WORKSPACE;
    if (!aligned_to(Wd, 2) || !aligned_to(X_nchw, 16) || !aligned_to(Y_nchw, 16) || !aligned_to(dev_status, 4) ||
        !aligned_to(workspace, 256))
        return MWU_ERR_ALIGNMENT;
    int sm_count = 0;
    const int rc = check_device(&sm_count);
    if (rc != MWU_OK) return rc;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    ConvParams p = {};
    p.g.all_live = 1;                                   // plain weights: no packed header to compare with
    p.g.N = rows;
    p.g.K = (long long)c * kh * kw;
    p.g.Y = Y_nchw;
    p.g.y_fp32 = y_dtype;
    p.g.dev_status = dev_status;
    const long long n_pad = (rows + kTileRows - 1) / kTileRows * kTileRows;
    unsigned short *xt = (unsigned short *)workspace;
    unsigned short *wd = (unsigned short *)((char *)workspace + x_bytes_aligned(n, c, h, w));
    const int taps = kh * kw;
    const long long K = p.g.K;
    return run_taps(p, X_nchw, n, c, h, w, kh, kw, pad, xt, wd, n_pad, sm_count, st,
                    [&](const unsigned short *x, unsigned short *xo, int HW, int tiles_hw, int tiles_c, unsigned n_tiles) {
        nchw_to_nhwc_kernel<<<n_tiles, PREP_THREADS, 0, st>>>(x, xo, c, HW, tiles_hw, tiles_c);
        const long long total = n_pad * K;
        const long long want = (total + 255) / 256, cap = (long long)sm_count * 16;
        permute_taps_kernel<<<(unsigned)(want < cap ? want : cap), 256, 0, st>>>((const unsigned short *)Wd, ldw, rows,
                                                                                  n_pad, taps, c, wd);
        count_launch(2);
    });
}
