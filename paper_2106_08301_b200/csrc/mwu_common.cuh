// Shared host/device helpers of the CUDA library: argument validation, the packed-format
// layout arithmetic, and small device utilities.  Nothing here is used by the CPU checker.
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stddef.h>

#include "mwu.h"

namespace mwu {

constexpr int kTileRows = 128;     // rows of W per packed record
constexpr int kStageK = 64;        // reduction-axis extent per packed record
constexpr int kHeaderBytes = 256;
constexpr size_t kAlign = 256;
constexpr unsigned long long kMagic = 0x314B43415055574Dull;   // "MWUPACK1" little-endian

inline size_t align_up(size_t x, size_t a = kAlign) { return (x + a - 1) / a * a; }

struct PackedLayout {
    int64_t n_pad, n_tiles, n_stages, n_unified, n_dense, n_pruned, n_plist;
    size_t off_rec, off_ulist, off_dpos, off_dpay, off_ppos, total;
};

// one entry of the record table: where the record starts in each class list
struct PackedRec { unsigned ubase, dbase, pbase, live; };

// Block shape of a descriptor (Section 3.1: 1-, 2- or 3-dim blocks).
struct ShapeInfo {
    int dk, dr, dt, taps;      // channels x rows x taps of a block; taps of the weight
    int64_t cin_groups;        // (cols / taps) / dk
    int64_t ntg;               // tap groups: ceil(taps / dt)
    int64_t mb;                // blocks
    bool shaped;               // false: blocks of `block` consecutive entries of one row
};

inline ShapeInfo shape_of(const mwu_proj_desc *d) {
    ShapeInfo s;
    s.dk = d->block;
    s.dr = d->block_rows > 1 ? d->block_rows : 1;
    s.dt = d->block_taps > 1 ? d->block_taps : 1;
    s.taps = d->taps > 1 ? d->taps : 1;
    s.shaped = s.dr > 1 || s.dt > 1 || s.taps > 1;
    s.ntg = (s.taps + s.dt - 1) / s.dt;
    s.cin_groups = s.dk > 0 ? (d->cols / s.taps) / s.dk : 0;
    s.mb = (d->rows / s.dr) * s.cin_groups * s.ntg;
    return s;
}

// A 2-dim shape whose blocks are runs of `block` entries in each of their rows can be packed: every
// such run becomes a 1-dim block with its block's class and magnitude.
inline bool packable(const ShapeInfo &s) { return s.dt == 1 && s.taps == 1; }

inline PackedLayout packed_layout(const mwu_proj_desc *d) {
    PackedLayout L;
    const ShapeInfo sh = shape_of(d);
    const int64_t mb = d->rows * d->cols / d->block;      // 1-dim runs (a block of dr rows makes dr of them)
    L.n_pad = (d->rows + kTileRows - 1) / kTileRows * kTileRows;
    L.n_tiles = L.n_pad / kTileRows;
    L.n_stages = d->cols / kStageK;
    L.n_pruned = d->k_prune * sh.dr;
    L.n_unified = (d->k_unify - d->k_prune) * sh.dr;
    L.n_dense = mb - d->k_unify * sh.dr;
    L.n_plist = L.n_pruned + (L.n_pad - d->rows) * (d->cols / d->block);
    L.off_rec = kHeaderBytes;
    L.off_ulist = align_up(L.off_rec + 16 * ((size_t)L.n_tiles * L.n_stages + 1));
    L.off_dpos = align_up(L.off_ulist + 8 * (size_t)L.n_unified);
    L.off_dpay = align_up(L.off_dpos + 2 * (size_t)L.n_dense);
    L.off_ppos = align_up(L.off_dpay + 2 * (size_t)d->block * L.n_dense);
    L.total = align_up(L.off_ppos + 2 * (size_t)L.n_plist);
    return L;
}

// MWU_OK or the error that describes what is wrong with the descriptor.
inline int validate_desc(const mwu_proj_desc *d, bool need_stage_multiple) {
    if (!d) return MWU_ERR_INVALID_ARG;
    if (d->rows <= 0 || d->cols <= 0) return MWU_ERR_SHAPE;
    if (d->block != 2 && d->block != 4 && d->block != 8 && d->block != 16) return MWU_ERR_SHAPE;
    if (d->cols % d->block != 0) return MWU_ERR_SHAPE;
    if (need_stage_multiple && d->cols % kStageK != 0) return MWU_ERR_SHAPE;
    if (d->block_rows < 0 || d->block_taps < 0 || d->taps < 0) return MWU_ERR_SHAPE;
    const ShapeInfo sh = shape_of(d);
    if (sh.shaped) {
        if (sh.dr != 1 && sh.dr != 2 && sh.dr != 4) return MWU_ERR_SHAPE;
        if (sh.dt != 1 && sh.dt != 2) return MWU_ERR_SHAPE;
        if (sh.dk * sh.dr * sh.dt > 16) return MWU_ERR_SHAPE;
        if (d->cols % sh.taps != 0 || (d->cols / sh.taps) % sh.dk != 0 || d->rows % sh.dr != 0) return MWU_ERR_SHAPE;
        if (d->prune_group_rows != 0 || d->prune_group_cols != 0) return MWU_ERR_SHAPE;   // groups: 1-dim blocks only
        if (need_stage_multiple && !packable(sh)) return MWU_ERR_SHAPE;   // no packed form: use Q with the dense entry points
    }
    if (d->prune_key != MWU_PRUNE_KEY_L2SQ && d->prune_key != MWU_PRUNE_KEY_L1)
        return MWU_ERR_INVALID_ARG;
    if (d->algo != MWU_ALGO_AUTO && d->algo != MWU_ALGO_ONE_PASS && d->algo != MWU_ALGO_MULTI_PASS)
        return MWU_ERR_INVALID_ARG;
    const int64_t mb = sh.mb;
    if (d->rows * d->cols / d->block >= (int64_t(1) << 31)) return MWU_ERR_SHAPE;
    if (d->k_prune < 0 || d->k_prune > d->k_unify || d->k_unify > mb) return MWU_ERR_SHAPE;
    if (d->prune_group_rows != 0 || d->prune_group_cols != 0) {
        const int gr = d->prune_group_rows, gc = d->prune_group_cols;
        if (gr != 32 && gr != 64 && gr != 128 && gr != 256) return MWU_ERR_SHAPE;
        if (gc != 16 && gc != 32 && gc != 64) return MWU_ERR_SHAPE;
        if (d->rows % gr != 0 || d->cols % gc != 0) return MWU_ERR_SHAPE;
        if (d->k_prune % ((int64_t)gr * gc / d->block) != 0) return MWU_ERR_SHAPE;   // whole groups only
    }
    return MWU_OK;
}

inline bool grouped(const mwu_proj_desc *d) { return d->prune_group_rows != 0; }

inline bool aligned_to(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

// MWU_OK when the current device is compute capability 10.x; also reports its SM count.
int check_device(int *sm_count);

// adds n to the process-wide count of kernels launched (mwu_kernel_launches)
void count_launch(int n = 1);

// 2- and 3-dim block shapes (mwu_shapes.cu)
namespace shapes {
size_t workspace_bytes(const mwu_proj_desc *desc);
int project(const mwu_proj_desc *desc, const float *W, const float *U_dual, float *Q, float *U_next,
            double *residual_sq, float *u, uint32_t *pruned_bitmap, uint32_t *unified_bitmap, uint32_t *sign_bits,
            double *loss_u, double *loss_p, uint32_t *dev_status, void *workspace, int sm_count, cudaStream_t st);
size_t lowering_bytes(const mwu_proj_desc *desc);
int lower(const mwu_proj_desc *desc, const float *u, const uint32_t *pruned_bitmap, const uint32_t *unified_bitmap,
          void *scratch, const float **u1, const uint32_t **pruned1, const uint32_t **unified1, int sm_count,
          cudaStream_t st);
}  // namespace shapes

}  // namespace mwu
