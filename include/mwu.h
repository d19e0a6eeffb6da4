/*
 * mwu.h -- C ABI of the micro-structured weight unification / pruning library
 *          (method of arXiv 2106.08301), CUDA, sm_100a only.
 *
 * Conventions that hold for every entry point
 *   - All tensor pointers are DEVICE pointers owned by the caller, 16-byte aligned unless
 *     stated otherwise; the library allocates nothing.  What it keeps between calls is host-side
 *     bookkeeping only: the address of one driver entry point, a launch counter
 *     (mwu_kernel_launches) and, for mwu_project_static, the device address of its built-in
 *     scratch array per device (stale after a cudaDeviceReset: do not call it again then).
 *   - Descriptors (mwu_proj_desc) and scalar arguments are HOST values.
 *   - Work is enqueued on `cuda_stream` (a cudaStream_t passed as void*, NULL = default
 *     stream).  No call synchronises with the host.
 *   - Argument errors are returned before anything is launched.  Conditions that only the
 *     device can see set bits in *dev_status (a device uint32_t the caller zeroes and reads
 *     after synchronising); outputs are then unspecified but every access stays in bounds.
 *   - There is no CPU fallback: on a device that is not compute capability 10.x the calls
 *     return MWU_ERR_UNSUPPORTED_DEVICE.
 *
 * Notation (paper, Section 3.1): a layer's weight tensor is viewed as W[rows][cols]
 * (rows = output features / filters, cols = the reduction axis; for a convolution
 * cols = cin*kh*kw in [cout, cin, kh, kw] order).  It is divided into Mb = rows*cols/block
 * micro-blocks of `block` consecutive entries of one row; block j = n*(cols/block) + kb
 * covers W[n][kb*block .. kb*block+block-1].
 */
#ifndef MWU_H_
#define MWU_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    MWU_OK = 0,
    MWU_ERR_INVALID_ARG = 1,        /* null pointer, negative size, unknown enum value        */
    MWU_ERR_SHAPE = 2,              /* cols % block != 0, block not in {2,4,8,16}, bad counts */
    MWU_ERR_ALIGNMENT = 3,          /* a pointer or leading dimension is not aligned          */
    MWU_ERR_WORKSPACE = 4,          /* workspace / packed buffer too small                    */
    MWU_ERR_UNSUPPORTED_DEVICE = 5, /* current device is not sm_100                           */
    MWU_ERR_CUDA = 6                /* a CUDA runtime or driver call failed                   */
} mwu_status;

/* bits of the device status word */
enum {
    MWU_DEV_NONFINITE = 1,  /* an input weight was NaN or Inf                                 */
    MWU_DEV_TIMEOUT = 2,    /* a bounded wait inside a kernel ran out                         */
    MWU_DEV_BOUNDS = 4,     /* packed data inconsistent with the descriptor (nothing written
                               out of bounds)                                                 */
    MWU_DEV_SELECT = 8      /* internal selection invariant violated                          */
};

typedef enum {
    MWU_PRUNE_KEY_L2SQ = 0, /* sum v^2: squared distance to the zero block (Eq. 7, q = 0)     */
    MWU_PRUNE_KEY_L1 = 1    /* sum |v|: the norm Section 3.1's pruning example names          */
} mwu_prune_key;

/* How mwu_project organises its kernels.  Every choice gives the same bits. */
typedef enum {
    MWU_ALGO_AUTO = 0,       /* one pass from 8192 blocks on, multi pass below                 */
    MWU_ALGO_ONE_PASS = 1,   /* outputs written in one sweep over W with thresholds estimated
                                from a sample, then the few blocks near a threshold corrected */
    MWU_ALGO_MULTI_PASS = 2  /* statistics pass, exact thresholds, emit pass                  */
} mwu_proj_algo;

typedef struct {
    int64_t rows, cols;     /* W[rows][cols], row-major, cols % block == 0                    */
    int32_t block;          /* micro-block width along cols: 2, 4, 8 or 16 (D1 of a 2- or
                               3-dim block shape, see block_rows / block_taps below)          */
    int32_t prune_key;      /* mwu_prune_key                                                  */
    int64_t k_unify;        /* number of blocks unified OR pruned (0 <= k_prune <= k_unify)   */
    int64_t k_prune;        /* number of blocks pruned to zero                                */
    int32_t algo;           /* mwu_proj_algo; read by mwu_project, mwu_project_static and
                               mwu_admm_step                                                  */
    int32_t block_rows;     /* D2: rows a block spans; 0 or 1 = blocks lie in one row, 2 or 4 */
    /* Grouped pruning (0, 0 = off: blocks are pruned one by one, the paper's rule).  When set,
     * the prune decision is taken for whole groups of prune_group_rows x prune_group_cols
     * weights: see mwu_project. */
    int32_t prune_group_rows;   /* 0, 32, 64, 128 or 256; rows % prune_group_rows == 0        */
    int32_t prune_group_cols;   /* 0, 16, 32 or 64; >= block; cols % prune_group_cols == 0    */
    /* 2- and 3-dim block shapes [D1, D2, D3] of Section 3.1 / Table 1 ([2,2], [2,2,2]) on a weight
     * viewed as W[rows][cin * taps] (taps = kh*kw, column = channel * taps + tap): a block spans
     * `block` input channels x block_rows rows x block_taps kernel taps.  Blocks are numbered
     * (row group, channel group, tap group), their weights ordered (row, channel, tap) for the
     * pairwise sums.  When block_taps does not divide taps the last tap group is shorter and its
     * blocks hold fewer weights (their unified value is the mean over the weights they hold).
     * block * block_rows * block_taps <= 16.  All zero (or one): the 1-dim blocks described above. */
    int32_t block_taps;     /* D3: kernel taps a block spans; 0 or 1, or 2                      */
    int32_t taps;           /* kh*kw of the weight (cols = cin * taps); 0 or 1 for a linear layer */
} mwu_proj_desc;

const char *mwu_status_string(int status);

/* Number of kernels this library has launched in this process so far (all entry points, all
 * threads).  Host-side counter, for telemetry. */
uint64_t mwu_kernel_launches(void);

/* Ratio -> integer count, (permille * n_blocks + 500) / 1000 in integers.  The paper gives
 * ratios (Section 1, "unification ratio"); counts cross this ABI as integers so that no
 * floating-point rounding can make caller and library disagree. */
int64_t mwu_count_from_permille(int64_t n_blocks, int32_t permille);

/*
 * mwu_project -- the Q-step of ADMM: Q = Unify(W + U)   (Algorithm 1; Eq. 7: a Euclidean
 * projection onto the set of tensors with k_prune zero blocks and k_unify - k_prune further
 * blocks whose entries share one absolute value).
 *
 * Per block (Section 3.1, Eq. 2 and the text after it) with v = W, or fp32(W + U_dual):
 *   q   = mean |v_l|                    unified value
 *   L_u = sum (|v_l| - q)^2             unification loss  (distance^2 to the unified block)
 *   L_p = sum v_l^2  (or sum |v_l|)     prune key         (distance^2 to the zero block)
 * evaluated in fp64, each operation rounded on its own, block sums as a balanced pairwise
 * tree.  Selection: the k_prune blocks with the smallest prune key are pruned; among the
 * others the k_unify - k_prune blocks with the smallest L_u are unified; equal keys are
 * ordered by block index.  Output of a pruned block is +0; of a unified block +q where
 * v_l >= 0 (this includes -0.0) and -q otherwise, q rounded to fp32; other blocks are
 * copied bit for bit.
 *
 * Grouped pruning (desc->prune_group_rows/cols set; not in the paper, whose Section 3.2 only says
 * that pruned blocks "can be completely skipped": a tensor-core tile can skip a column slice only
 * when it is zero in all of the tile's rows, so this variant prunes whole tile-aligned groups).
 * The tensor is cut into groups of prune_group_rows x prune_group_cols weights; a group's key is
 * the sum of its blocks' prune keys (per row a pairwise tree over the row's blocks inside the
 * group, then a pairwise tree over the group's rows, fp64); the k_prune / (blocks per group)
 * groups with the smallest keys are zeroed (equal keys: lower group index, row tile first);
 * k_prune must be a multiple of the blocks per group.  This is the Euclidean projection onto
 * "at least that many groups are zero".  Unification then works block by block as above among
 * the blocks outside the pruned groups.
 *
 *   W, U_dual      in   fp32 [rows*cols]; U_dual may be NULL
 *   Q              out  fp32 [rows*cols]; may be NULL (only the compressed form is wanted)
 *   u              out  fp32 [Mb]: fp32(q) for unified blocks, +0 otherwise
 *   pruned_bitmap, unified_bitmap
 *                  out  uint32 [ceil(Mb/32)], bit (j%32) of word (j/32); unused bits 0
 *   sign_bits      out  uint32 [ceil(rows*cols/32)], bit = (v_l < 0) for every weight
 *   loss_u, loss_p out  fp64 [Mb] each, may be NULL: L_u and the prune key of every block
 *   dev_status     i/o  device uint32, bits OR-ed in
 *   workspace      device scratch of at least mwu_project_workspace_bytes(desc) bytes,
 *                  256-byte aligned; contents undefined on entry and exit
 * Errors: MWU_ERR_* as listed above; nothing is launched on error.
 */
size_t mwu_project_workspace_bytes(const mwu_proj_desc *desc);
int mwu_project(const mwu_proj_desc *desc, const float *W, const float *U_dual, float *Q,
                float *u, uint32_t *pruned_bitmap, uint32_t *unified_bitmap,
                uint32_t *sign_bits, double *loss_u, double *loss_p, uint32_t *dev_status,
                void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * mwu_admm_step -- the Q-step and the dual step of one ADMM iteration in one sweep
 * (Algorithm 1: Q = Unify(W + U), then U <- U + W - Q; the dual update is the last of the three
 * ADMM steps of Section 3.3, and ||W - Q + U||_F^2 is the quadratic term of the augmented
 * Lagrangian given there, without its factor rho/2).
 *
 * With v = W, or fp32(W + U_dual), and Q as mwu_project computes it:
 *   U_next[l]    = fp32(v_l - Q_l)       one subtraction per entry: v_l for a pruned block,
 *                                        +0 for a block that keeps its values
 *   residual_sq  = sum over pruned blocks of sum v_l^2 + sum over unified blocks of L_u
 *                = ||v - Q||_F^2 with the unified magnitudes unrounded, accumulated in fp64
 *                  (the order of the additions is not fixed: expect the last bits to vary)
 * rho * U_next is also the gradient of the quadratic term with respect to W, which the caller's
 * optimiser needs for the next W-step.
 *
 *   U_next        out  fp32 [rows*cols]; may be NULL.  Must not overlap W or U_dual (they are read
 *                      again after U_next has been written): MWU_ERR_INVALID_ARG
 *   residual_sq   out  device fp64 [1], 8-byte aligned; may be NULL; zeroed by the call
 *   At least one of the two must be given.  All other arguments, outputs, workspace and errors as
 *   mwu_project (without the per-block loss outputs).
 */
int mwu_admm_step(const mwu_proj_desc *desc, const float *W, const float *U_dual, float *Q,
                  float *U_next, double *residual_sq, float *u, uint32_t *pruned_bitmap,
                  uint32_t *unified_bitmap, uint32_t *sign_bits, uint32_t *dev_status,
                  void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * mwu_project_static -- mwu_project without a caller-supplied workspace.  (The paper has no
 * counterpart: this is a packaging variant of the same projection, with the same outputs.)
 *
 * For callers that cannot allocate device memory where they need the projection -- code running
 * inside an engine that owns the memory pool, or after a job's memory budget has been frozen,
 * where a cudaMalloc may fail or stall the device.  The scratch memory is a fixed array inside
 * the library's device image (about 8 MB, held by every GPU that loads the library until the
 * process exits), so the call allocates nothing.
 *
 * Limits and rules:
 *   - at most MWU_STATIC_MAX_BLOCKS blocks (rows*cols/block); larger tensors return
 *     MWU_ERR_WORKSPACE and nothing is launched -- use mwu_project with your own workspace;
 *   - the first call on each device looks up the device address of the built-in array.  If the
 *     library's device code has not been loaded on that device yet, this query loads it, and the
 *     driver then sets the array's memory aside; so make that first call at start-up, before a
 *     memory budget is frozen and outside any stream capture.  Later calls on the device change
 *     nothing;
 *   - all calls on one device share the array: two calls whose kernels can overlap on the GPU
 *     (different streams without an ordering between them) race and give undefined results;
 *     calls on one stream, or otherwise ordered, are fine.  Each call clears the part of the
 *     scratch that must start at zero, so earlier calls leave no trace.
 * Arguments, outputs and errors are those of mwu_project.
 */
#define MWU_STATIC_MAX_BLOCKS 1048576
int mwu_project_static(const mwu_proj_desc *desc, const float *W, const float *U_dual, float *Q,
                       float *u, uint32_t *pruned_bitmap, uint32_t *unified_bitmap,
                       uint32_t *sign_bits, double *loss_u, double *loss_p, uint32_t *dev_status,
                       void *cuda_stream);

/*
 * mwu_pack -- the storage form of Section 3.1 / Table 1: a unified block keeps one
 * magnitude, a pruned block nothing, every weight one sign bit, the remaining blocks their
 * values (here rounded to bf16, the type the GEMM multiplies in).
 *
 * Needs cols % 64 == 0.  Inputs are mwu_project's inputs and outputs for the same desc.
 * `packed` receives exactly mwu_packed_bytes(desc) bytes (256-byte aligned buffer).  A record is
 * a row tile of 128 rows x 64 columns; it has 128 * 64/block block slots, numbered
 * pos = row_in_tile * (64/block) + block_in_record.  A block is addressed by `off`, the byte
 * offset of its first value in the record's decoded bf16 tile as the GEMM lays it out in shared
 * memory: row r starts at (r/8)*1024 + (r%8)*128 and its 16-byte chunk c sits at chunk position
 * c ^ (r%8).  Per record the blocks are listed by class, records in tile-major order.  Inside
 * a class list the entries are dealt round-robin over the store slots
 * slot = (off % 128) / min(2*block, 16): entries of one slot keep ascending pos order, and the
 * list takes the first entry of every slot (ascending slot), then the second of every slot that
 * has one, and so on, so that neighbouring entries fall into different shared-memory banks:
 *   header  256 B : u64 magic "MWUPACK1", version 4, rows, cols, block, rows_padded, n_tiles,
 *                   n_stages, n_pruned, n_unified, n_dense, n_plist, byte offsets of rec, ulist,
 *                   dpos, dpay, ppos, total bytes
 *   rec     16 B per record plus one closing entry: u32 ubase, dbase, pbase (index of the
 *                   record's first entry in ulist, dpos/dpay, ppos; the closing entry holds the
 *                   totals), u32 live (bit s set if some row has a non-pruned block overlapping
 *                   columns [16s,16s+16) of the record)
 *   ulist   8 B per unified block: u32 sign bits, weight l at bit l/2 + 16*(l%2) (set when
 *                   v_l < 0); u16 off; u16 bf16(unified value), round to nearest even
 *   dpos    u16 off per remaining non-pruned ("dense") block
 *   dpay    the dense block's `block` values as bf16 (round to nearest even), same order
 *   ppos    u16 off per pruned block
 * Rows beyond `rows` up to the next multiple of 128 are padding and are listed as pruned
 * (n_plist = n_pruned + padding blocks).  Sections start on 256-byte boundaries, gaps are
 * zero.  A mismatch between the bitmaps and desc's counts sets MWU_DEV_BOUNDS.
 */
size_t mwu_packed_bytes(const mwu_proj_desc *desc);
int mwu_pack(const mwu_proj_desc *desc, const float *W, const float *U_dual, const float *u,
             const uint32_t *pruned_bitmap, const uint32_t *unified_bitmap,
             const uint32_t *sign_bits, void *packed, size_t packed_bytes,
             uint32_t *dev_status, void *cuda_stream);

/*
 * mwu_gemm -- layer forward on the compressed weights (Section 3.2): Y = X . W_hat^T with
 * W_hat decoded from `packed` (0 for pruned blocks, +-bf16(u) by sign bit for unified blocks,
 * the stored bf16 values otherwise).  Column slices that are pruned in every row of a weight
 * tile are skipped; products are bf16 x bf16 accumulated in fp32.
 *
 *   X        in   bf16 [M][ldx], ldx >= cols, ldx % 8 == 0
 *   Y        out  [M][ldy], ldy >= rows; y_dtype 0: bf16 (round to nearest even, ldy % 8 == 0),
 *                 1: fp32 (ldy % 4 == 0)
 * M may be any positive value (ragged last tile is handled); M == 0 is a no-op.
 * `desc` must be the descriptor `packed` was made with (the host cannot read the device buffer):
 * the kernels compare it with the header of `packed` and, on a mismatch, set MWU_DEV_BOUNDS and
 * write nothing.  The same holds for mwu_decode, mwu_gemm_ws and mwu_conv_implicit.
 */
int mwu_gemm(const mwu_proj_desc *desc, const void *packed, const void *X, int64_t M,
             int64_t ldx, void *Y, int64_t ldy, int32_t y_dtype, uint32_t *dev_status,
             void *cuda_stream);

/*
 * mwu_decode -- the compressed weights expanded to a dense matrix (Section 3.2, the layer's
 * weight as the GEMM sees it): Wd[r][c] = W_hat[r][c] in bf16, i.e. 0 for pruned blocks,
 * +-bf16(u) by sign bit for unified blocks, the stored bf16 value otherwise.
 *
 *   Wd   out  device, bf16 [n_pad][ldw] with n_pad = rows rounded up to a multiple of 128,
 *             ldw >= cols, ldw % 8 == 0, 16-byte aligned; rows past `rows` are written as zeros.
 * Every element of the n_pad x cols region is written; the caller owns the buffer.
 */
int mwu_decode(const mwu_proj_desc *desc, const void *packed, void *Wd, int64_t ldw,
               uint32_t *dev_status, void *cuda_stream);

/*
 * mwu_gemm_ws -- mwu_gemm with a caller-owned scratch buffer.  With many activation rows the
 * fused kernel would decode every weight record once per 512-row activation tile; given
 * `workspace` of at least mwu_gemm_workspace_bytes(desc, M) bytes (device memory, 256-byte
 * aligned) the weights are expanded once per call as by mwu_decode and a two-operand
 * tensor-core GEMM reads them, still skipping the column slices that are pruned in every row
 * of a weight tile.  The result is the same contraction with the same rounding of operands
 * (bf16 x bf16, fp32 accumulation); only the summation order inside the tensor cores may differ.
 * mwu_gemm_workspace_bytes returns 0 when M is too small for this to pay (or desc is invalid);
 * with workspace == NULL, or fewer bytes than that, the call behaves exactly like mwu_gemm.
 * The workspace holds nothing between calls and may be shared by calls on the same stream.
 */
size_t mwu_gemm_workspace_bytes(const mwu_proj_desc *desc, int64_t M);
int mwu_gemm_ws(const mwu_proj_desc *desc, const void *packed, const void *X, int64_t M,
                int64_t ldx, void *Y, int64_t ldy, int32_t y_dtype, void *workspace,
                size_t workspace_bytes, uint32_t *dev_status, void *cuda_stream);

/*
 * mwu_conv_implicit -- the same contraction for a convolution lowered to GEMM without
 * materialising the lowered matrix (Section 3.2 treats a layer's convolution as a GEMM):
 *   A[(n,oh,ow)][(c,i,j)] = x[n][c][oh*stride+i-pad][ow*stride+j-pad]  (0 outside),
 *   y[n][o][oh][ow] = sum_k A[(n,oh,ow)][k] * W_hat[o][k],  desc->cols == c*kh*kw.
 *   X  in  bf16 NCHW [n][c][h][w];   Y  out NCHW [n][rows][oh][ow], y_dtype as above.
 */
int mwu_conv_implicit(const mwu_proj_desc *desc, const void *packed, const void *X_nchw,
                      int32_t n, int32_t c, int32_t h, int32_t w, int32_t kh, int32_t kw,
                      int32_t stride, int32_t pad, void *Y_nchw, int32_t y_dtype,
                      uint32_t *dev_status, void *cuda_stream);

/*
 * mwu_conv_implicit_ws -- mwu_conv_implicit with a caller-owned scratch buffer, the counterpart
 * of mwu_gemm_ws: given `workspace` of at least mwu_conv_workspace_bytes(...) bytes (device
 * memory, 256-byte aligned) the weights are expanded once per call as by mwu_decode and the
 * tensor-core kernel reads them beside the gathered activation tiles, instead of decoding every
 * weight record again for every activation tile.  Same contraction, same rounding of operands.
 * mwu_conv_workspace_bytes returns 0 when the shape is not served by this path (or desc is
 * invalid); with workspace == NULL, or fewer bytes than that, the call behaves exactly like
 * mwu_conv_implicit.  The workspace holds nothing between calls.
 */
size_t mwu_conv_workspace_bytes(const mwu_proj_desc *desc, int32_t n, int32_t c, int32_t h,
                                int32_t w, int32_t kh, int32_t kw, int32_t stride, int32_t pad);
int mwu_conv_implicit_ws(const mwu_proj_desc *desc, const void *packed, const void *X_nchw,
                         int32_t n, int32_t c, int32_t h, int32_t w, int32_t kh, int32_t kw,
                         int32_t stride, int32_t pad, void *Y_nchw, int32_t y_dtype,
                         void *workspace, size_t workspace_bytes, uint32_t *dev_status,
                         void *cuda_stream);

/*
 * mwu_keep_n_of_m -- the in-block pruning of Section 4.7 (the pruning half of the paper's
 * combination test: 1x4 blocks with half of every block pruned, the pattern sparse tensor cores
 * accept).  Of every m = 4 consecutive entries of a row of v = W, or fp32(W + U_dual), the n with
 * the largest magnitude are kept (equal magnitudes: the lower index) and the others become +0:
 * the Euclidean projection (Eq. 7) onto "at most n non-zeros in every group of m".
 *
 *   W, U_dual   in   fp32 [rows*cols], cols % 4 == 0; U_dual may be NULL
 *   Q           out  fp32 [rows*cols]; may be NULL
 *   keep_bits   out  uint32 [ceil(rows*cols/32)], bit (f%32) of word (f/32) set when weight f is kept
 *   Wd          out  bf16 [rows][ldw], ldw >= cols, ldw % 8 == 0; may be NULL: Q rounded to bf16, the
 *                    weight matrix mwu_gemm_dense multiplies with
 * Only m == 4 is built (n = 0..4): MWU_ERR_SHAPE otherwise.  A non-finite input sets
 * MWU_DEV_NONFINITE.
 */
int mwu_keep_n_of_m(int64_t rows, int64_t cols, int32_t n, int32_t m, const float *W,
                    const float *U_dual, float *Q, uint32_t *keep_bits, void *Wd, int64_t ldw,
                    uint32_t *dev_status, void *cuda_stream);

/*
 * mwu_gemm_dense -- Y = X . Wd^T for a plain bf16 weight matrix Wd[rows][ldw] (Section 3.2's layer
 * forward for weights that carry no block classes, e.g. the output of mwu_keep_n_of_m or of
 * mwu_decode): the two-operand tensor-core kernel behind mwu_gemm_ws, bf16 x bf16 accumulated in
 * fp32.  X, Y, M, ldx, ldy, y_dtype as mwu_gemm; ldw >= cols, ldw % 8 == 0.  The kept / dropped
 * pattern of mwu_keep_n_of_m saves storage only: every product is executed.
 */
int mwu_gemm_dense(int64_t rows, int64_t cols, const void *Wd, int64_t ldw, const void *X, int64_t M,
                   int64_t ldx, void *Y, int64_t ldy, int32_t y_dtype, uint32_t *dev_status,
                   void *cuda_stream);

/*
 * mwu_conv_dense -- the convolution of mwu_conv_implicit for a plain bf16 weight matrix
 * Wd[rows][ldw] whose first c*kh*kw columns are in [c][kh][kw] order (the counterpart of
 * mwu_gemm_dense; it serves the block shapes that have no packed form: project with Q, round Q to
 * bf16, multiply).  Shapes: stride 1, c % 64 == 0, at most 128 output pixels per row;
 * mwu_conv_dense_workspace_bytes returns 0 for any other shape and the call then returns
 * MWU_ERR_SHAPE.  `workspace`: device memory of that many bytes, 256-byte aligned, holding nothing
 * between calls.
 */
size_t mwu_conv_dense_workspace_bytes(int64_t rows, int32_t n, int32_t c, int32_t h, int32_t w,
                                      int32_t kh, int32_t kw, int32_t stride, int32_t pad);
int mwu_conv_dense(int64_t rows, const void *Wd, int64_t ldw, const void *X_nchw, int32_t n, int32_t c,
                   int32_t h, int32_t w, int32_t kh, int32_t kw, int32_t stride, int32_t pad,
                   void *Y_nchw, int32_t y_dtype, void *workspace, size_t workspace_bytes,
                   uint32_t *dev_status, void *cuda_stream);

/*
 * mwu_debug_conv_wait -- testing aid for the bounded waits inside the kernels (the paper has no
 * counterpart).  Every wait of a kernel on one of its own barriers has a limit, after which the
 * kernel sets MWU_DEV_TIMEOUT in *dev_status, lets the copies it has in flight land, releases its
 * tensor memory and returns, leaving the context usable.  This call makes that path observable on
 * the tensor-core kernel of mwu_conv_implicit_ws: `limit_cycles` replaces the limit (about two
 * seconds by default; <= 0 restores it) and `withhold_stage` names the running number of one
 * pipeline stage whose loads the producer leaves out in every CTA, so that the consumer's wait for
 * it must run out (-1: none).  Process-wide host setting, read when mwu_conv_implicit_ws is called;
 * not meant for production code.
 */
void mwu_debug_conv_wait(int64_t limit_cycles, int64_t withhold_stage);

#ifdef __cplusplus
}
#endif
#endif /* MWU_H_ */
