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

inline PackedLayout packed_layout(const mwu_proj_desc *d) {
    PackedLayout L;
    const int64_t mb = d->rows * d->cols / d->block;
    L.n_pad = (d->rows + kTileRows - 1) / kTileRows * kTileRows;
    L.n_tiles = L.n_pad / kTileRows;
    L.n_stages = d->cols / kStageK;
    L.n_pruned = d->k_prune;
    L.n_unified = d->k_unify - d->k_prune;
    L.n_dense = mb - d->k_unify;
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
    if (d->prune_key != MWU_PRUNE_KEY_L2SQ && d->prune_key != MWU_PRUNE_KEY_L1)
        return MWU_ERR_INVALID_ARG;
    if (d->algo != MWU_ALGO_AUTO && d->algo != MWU_ALGO_ONE_PASS && d->algo != MWU_ALGO_MULTI_PASS)
        return MWU_ERR_INVALID_ARG;
    const int64_t mb = d->rows * d->cols / d->block;
    if (mb >= (int64_t(1) << 31)) return MWU_ERR_SHAPE;
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

}  // namespace mwu
