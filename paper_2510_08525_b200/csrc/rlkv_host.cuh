// Host-side helpers shared by the two cache objects of librlkv (the lock-step cache of rlkv_api.cu
// and the paged, ragged cache of rlkv_paged.cu).
#pragma once

#include <stdint.h>
#include <stdio.h>

#include "../../include/rlkv.h"
#include "rlkv_internal.cuh"

namespace rlkv {

extern thread_local char g_cuda_text[256];  // text behind RLKV_ECUDA for rlkv_strerror (rlkv_api.cu)

inline int cuda_fail(cudaError_t e, const char* what)
{
    snprintf(g_cuda_text, sizeof g_cuda_text, "CUDA error in %s: %s", what, cudaGetErrorString(e));
    return RLKV_ECUDA;
}
#define RLKV_CUDA(call)                                  \
    do {                                                 \
        cudaError_t e_ = (call);                         \
        if (e_ != cudaSuccess) return ::rlkv::cuda_fail(e_, #call); \
    } while (0)

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

constexpr int kMaxGridSms = 160;  // scratch is sized for 2 CTAs on each of up to 160 SMs
constexpr int kMinItemTiles = 2;  // smallest work item of the decode kernel (sizes the scratch)

// Most partial records a decode launch of this shape can write, over every length up to tf tiles
// per full unit and every grid up to max_grid CTAs.
inline long long most_slots(int U, int tf, int Uc, int tc, int max_grid)
{
    long long most = 0;
    for (int p = 1; p <= max_grid; ++p) {
        const long long m = max_slots(U, tf, Uc, tc, p, kMinItemTiles);
        if (m > most) most = m;
    }
    return most;
}

// Most pipeline stages (<= 8) that fit `ctas_per_sm` CTAs of the decode kernel on one SM
// (228 KB per SM, 1 KB of it reserved per resident CTA).  The stage count is a multiple of the
// number of consumer groups, so that a given stage is always consumed by the same group: an
// mbarrier parity wait can only tell two phases apart, and a group that reached a stage a whole
// phase early would take the wait for the phase before as satisfied.
inline int max_stages(int head_dim, int group, int groups, int ctas_per_sm, int mode = kModePlain)
{
    for (int st = 8; st >= 2; --st) {
        if (st % groups != 0) continue;
        const size_t one = decode_smem_bytes(head_dim, st, group, groups, mode);
        if (one <= (size_t)kMaxDynamicSmem && (one + 1024) * ctas_per_sm <= 228u * 1024u) return st;
    }
    return 0;
}

// How the decode launches of one step follow one another in the stream.  Consecutive launches use
// different copies of the split-KV scratch (partial records, claim counter, and in the paged cache the
// tickets), so launch l may run beside launch l-1; it shares its copy with launch l-2 and must not start
// before that one has completed.  The device guarantees it: a launch is started in one of three ways,
//   ordinary   (overlap 0, dep_wait 0): it starts when everything before it in the stream has completed,
//              and lets its successor start at once;
//   dep_wait 1 (the launch right after the step's append launch): it may start beside the append launch,
//              waits for it before it touches what that launch writes, and only then lets its successor
//              start;
//   dep_wait 2 (every other launch): it may start beside its predecessor; an otherwise idle thread of
//              each of its CTAs waits (griddepcontrol.wait) until the predecessor has completed and only
//              then executes griddepcontrol.launch_dependents.
// A launch with the programmatic-serialization attribute starts once every CTA of its predecessor has
// executed launch_dependents or exited; in all three cases that happens only after the predecessor's own
// predecessor has completed.  So at most two decode launches are ever in flight and launch l never runs
// beside launch l-2, however the block scheduler places CTAs.
// `first`: the first decode launch of this run of launches; `after_append`: it directly follows the
// step's append launch in the stream (otherwise something else precedes it, e.g. a wait for a copy).
struct StepLaunchMode {
    bool overlap;
    int dep_wait;
};
inline StepLaunchMode step_launch_mode(bool first, bool after_append)
{
    if (!first) return StepLaunchMode{true, 2};
    if (after_append) return StepLaunchMode{true, 1};
    return StepLaunchMode{false, 0};
}

constexpr int kDefaultItemTiles = 32;  // largest "smallest work item" of launches that overlap or span a whole step

// The schedule of a whole step in one launch: U full units of tf tiles and Uc compressed units of tc
// tiles over all layers, for `grid` CTAs.  The full units go to the whole-unit prefix (one static item
// per CTA, units streamed in one piece: no partial records, no merges) except for as many as give
// every CTA about six items to claim, so that CTAs on a slower path to memory end together with the
// others (measured: CTAs differ by about 1 % in the tiles they get through; with a third of the units
// left to claim, as at first, the step was 1 % slower -- every claimed unit is cut into 4-5 pieces).
// `prefix` false: no whole-unit prefix, every item is claimed.  `unit_items`: the prefix is claimed unit
// by unit (a paged batch of unequal lengths: equal tile ranges would hold unequal numbers of tiles that
// exist, whole units can still be streamed in one piece).
inline Schedule step_schedule(int U, int tf, int Uc, int tc, int grid, int item_most, bool prefix = true,
                              long long real_tiles = -1, bool unit_items = false)
{
    // (paged cache: `real_tiles` of the tiles exist, and they decide the item size)
    const long long all_tiles = real_tiles >= 0 ? real_tiles : (long long)U * tf + (long long)Uc * tc;
    int item_tiles = (int)(all_tiles / grid);
    if (item_tiles > item_most) item_tiles = item_most;
    if (item_tiles < kMinItemTiles) item_tiles = kMinItemTiles;
    int U0 = 0;
    if (U > 0 && prefix) {
        long long rest_wanted = 6ll * grid * item_tiles;  // tiles left to the claimed items
        const long long flat_tiles = (long long)U * tf + (long long)Uc * tc;
        if (real_tiles > 0 && real_tiles < flat_tiles) rest_wanted = rest_wanted * flat_tiles / real_tiles;  // ... that exist
        long long most = U - (rest_wanted - (long long)Uc * tc + tf - 1) / tf;
        if (most > U) most = U;
        U0 = most > 0 ? (int)most : 0;
    }
    return make_schedule(U, tf, Uc, tc, grid, item_tiles, U0, 0, unit_items);
}

}  // namespace rlkv
struct rlkv_paged;
namespace rlkv {
// Internal entry points of the paged cache for the lock-step cache kept in 8 bits (rlkv_api.cu).
int paged_prefill_strided(rlkv_paged* p, int layer, int slot, const void* k, const void* v, int n_tokens,
                          long long entry_stride, void* stream);
uint64_t paged_launch_count(const rlkv_paged* p);

struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev)
    {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
        if (prev == dev) prev = -1;
    }
    ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};

// Tensor map over a pool of `rows` rows of head_dim bf16 at `base`, boxes of one 64-row tile.
// The pool is described as rows of 128-byte pieces so that one box is one contiguous run of memory
// and still obeys the 128-byte limit of the swizzled inner dimension.  For head_dim 128 the two
// halves of the rows are the OUTER dimension of the box, so the tile lands in shared memory as two
// blocks of [64 rows][128 bytes]: eight consecutive rows of a block are then eight different
// swizzle phases (with 256-byte rows only four, and every ldmatrix would take a two-way bank
// conflict).
//   head_dim 128: [2 halves][rows][64]  box [2][64 rows][64]  (16 KB)
//   head_dim  64: [rows][64]            box [64 rows][64]     ( 8 KB)
inline int encode_pool_tensor_map(CUtensorMap* tmap, void* base, long long rows, int head_dim)
{
    typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                      const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                      CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    RLKV_CUDA(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q));
    if (!fn || q != cudaDriverEntryPointSuccess) return cuda_fail(cudaErrorNotSupported, "cuTensorMapEncodeTiled lookup");
    CUresult r;
    const CUtensorMapL2promotion l2p = CU_TENSOR_MAP_L2_PROMOTION_L2_256B;
    if (head_dim == 128) {
        const cuuint64_t dims[3] = {64, (cuuint64_t)rows, 2};
        const cuuint64_t strides[2] = {256, 128};
        const cuuint32_t box[3] = {64, (cuuint32_t)kTile, 2};
        const cuuint32_t estr[3] = {1, 1, 1};
        r = reinterpret_cast<EncodeTiledFn>(fn)(tmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, base, dims, strides, box, estr,
                                                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, l2p,
                                                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    } else {
        const cuuint64_t dims[2] = {64, (cuuint64_t)rows};
        const cuuint64_t strides[1] = {128};
        const cuuint32_t box[2] = {64, (cuuint32_t)kTile};
        const cuuint32_t estr[2] = {1, 1};
        r = reinterpret_cast<EncodeTiledFn>(fn)(tmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, base, dims, strides, box, estr,
                                                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, l2p,
                                                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    }
    if (r != CUDA_SUCCESS) {
        snprintf(g_cuda_text, sizeof g_cuda_text, "cuTensorMapEncodeTiled failed with CUresult %d", (int)r);
        return RLKV_ECUDA;
    }
    return RLKV_OK;
}

// Tensor map over `rows` rows of row_bytes (64 or 128) bytes at `base`, boxes of box_rows whole rows,
// swizzled over the row width: the view of the paged cache's 8-bit pool (128-byte rows, a page per box).
inline int encode_byte_rows_tensor_map(CUtensorMap* tmap, void* base, int row_bytes, long long rows, int box_rows)
{
    typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                      const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                      CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    RLKV_CUDA(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q));
    if (!fn || q != cudaDriverEntryPointSuccess) return cuda_fail(cudaErrorNotSupported, "cuTensorMapEncodeTiled lookup");
    const cuuint64_t dims[2] = {(cuuint64_t)row_bytes, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)row_bytes};
    const cuuint32_t box[2] = {(cuuint32_t)row_bytes, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = reinterpret_cast<EncodeTiledFn>(fn)(
        tmap, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
        row_bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        snprintf(g_cuda_text, sizeof g_cuda_text, "cuTensorMapEncodeTiled (8-bit pool) failed with CUresult %d", (int)r);
        return RLKV_ECUDA;
    }
    return RLKV_OK;
}

}  // namespace rlkv
