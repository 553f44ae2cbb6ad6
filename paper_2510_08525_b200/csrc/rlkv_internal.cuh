// Internal definitions shared by the host API and the kernels of librlkv.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace rlkv {

constexpr int kTile = 64;        // tokens per K/V tile (one pipeline stage holds a K and a V tile)
constexpr int kMaxGroup = 8;     // query heads per KV head handled by one tile pass
constexpr int kGroupWarps = 4;   // consumer warps that share one tile (16 tokens each)
constexpr int kMaxConsumerGroups = 3;
constexpr int kMaxDynamicSmem = 227 * 1024;
constexpr int kMergePad = 4;     // floats of padding per head row in the cross-warp merge area

// Kernel status codes (device error word).
enum : int {
    kStatusOk = 0,
    kStatusFullWaitTimeout = 1,   // a consumer gave up waiting for a tile to land
    kStatusEmptyWaitTimeout = 2,  // the producer gave up waiting for a stage to be released
    kStatusDrainTimeout = 3       // the producer gave up waiting for its own copies in flight
};

// One (cta, slot) record of split-KV partial results: running max and sum (log2 domain) and the
// un-normalised output rows of the kMaxGroup query heads of the unit.
__host__ __device__ constexpr int partial_floats(int head_dim) {
    return 2 * kMaxGroup + kMaxGroup * head_dim;
}

// Everything a decode launch needs about one layer.  Passed by value.
struct DecodeArgs {
    const __nv_bfloat16* pool;  // base of the row pool, rows of head_dim bf16
    long long full_row0;        // first pool row of the layer's full-head region
    long long comp_row0;        // first pool row of the layer's compressed-head region
    const int* head_of_slot;    // [kv_heads]: KV head of full slot 0..n_full-1, then of comp slots
    const __nv_bfloat16* q;     // [batch][q_heads][head_dim]
    float* out;                 // [batch][q_heads][head_dim]
    float* partials;            // [grid][2][partial_floats]
    int* tickets;               // [batch*n_full] for this layer, zero between launches
    int* status;                // device error word
    unsigned long long* timeline;  // debug: [grid][4] globaltimer stamps
    int n_full, n_comp;         // heads of each class in this layer
    int rows_full, rows_comp;   // allocated rows per head (multiples of kTile)
    int len_full, len_comp;     // valid rows per head right now: n and min(n, sink+window)
    int batch, group, q_heads;
    int tiles_full, tiles_comp; // ceil(len / kTile) per head of each class
    int full_tiles;             // batch*n_full*tiles_full: the flat tile space of the full units
    int grid_full;              // CTAs that share the full tiles (<= grid, <= full_tiles)
    int comp_units;             // batch*n_comp
    float scale_log2;           // log2(e) / sqrt(head_dim)
    int debug;
};

struct AppendArgs {
    __nv_bfloat16* pool;
    long long full_row0, comp_row0;
    const int* slot_of_head;    // [kv_heads]: >= 0 full slot, < 0: -(comp slot + 1)
    const __nv_bfloat16* k;     // [n_tokens][batch][kv_heads][head_dim]
    const __nv_bfloat16* v;
    int n_full, n_comp, rows_full, rows_comp;
    int batch, kv_heads, head_dim;
    int t0, n_tokens;           // tokens t0 .. t0+n_tokens-1 are appended
    int sink, window;
};

// ---- work decomposition -------------------------------------------------------------------------
// Units are (batch row, head-of-class).  The tiles of the FULL units form one flat space of
// full_tiles = batch*n_full*tiles_full tiles (unit u owns tiles [u*tiles_full, (u+1)*tiles_full));
// CTA c < grid_full owns the flat range [c*T/Pf, (c+1)*T/Pf), so a long scan may be split across
// CTAs.  COMPRESSED units are short (sink + ring rows): they are never split; CTA c of P owns the
// units [c*UC/P, (c+1)*UC/P).  A CTA walks its compressed units first, then its full range.

struct UnitInfo {
    int unit;        // index inside its class
    int tile;        // tile index inside the unit
    int tiles;       // tiles of the unit
    int len;         // valid rows of the unit
    int b, head;     // batch row, KV head
    long long krow;  // pool row of the unit's K row 0 (V rows start `rows` later)
    int rows;        // allocated rows per K (and per V) of the unit
    int first_tile;  // flat index of the unit's tile 0 (full units only)
    bool full;
};

__host__ __device__ inline long long cta_start(int c, int T, int P) {
    return ((long long)c * T) / P;
}
// The CTA whose range contains flat tile x: the largest c with c*T/P <= x (needs P <= T).
__host__ __device__ inline int cta_of_tile(long long x, int T, int P) {
    return (int)(((x + 1) * P - 1) / T);
}

// A CTA's share of the work.
struct CtaWork {
    int cu0, cu1;     // compressed units [cu0, cu1)
    int f0, f1;       // flat full tiles [f0, f1)
    int comp_tiles;   // (cu1 - cu0) * tiles_comp
    int total;        // comp_tiles + f1 - f0: the CTA's tiles, in processing order
};

__device__ inline CtaWork cta_work(const DecodeArgs& a, int c, int P) {
    CtaWork w;
    w.cu0 = (int)cta_start(c, a.comp_units, P);
    w.cu1 = (int)cta_start(c + 1, a.comp_units, P);
    w.f0 = c < a.grid_full ? (int)cta_start(c, a.full_tiles, a.grid_full) : 0;
    w.f1 = c < a.grid_full ? (int)cta_start(c + 1, a.full_tiles, a.grid_full) : 0;
    w.comp_tiles = (w.cu1 - w.cu0) * a.tiles_comp;
    w.total = w.comp_tiles + (w.f1 - w.f0);
    return w;
}

// The unit and tile behind position v of a CTA's tile sequence.
__device__ inline UnitInfo locate(const DecodeArgs& a, const CtaWork& w, int v) {
    UnitInfo u;
    if (v < w.comp_tiles) {
        const int k = v / a.tiles_comp;
        u.unit = w.cu0 + k;
        u.tile = v - k * a.tiles_comp;
        u.tiles = a.tiles_comp;
        u.len = a.len_comp;
        u.b = u.unit / a.n_comp;
        u.head = a.head_of_slot[a.n_full + (u.unit - u.b * a.n_comp)];
        u.rows = a.rows_comp;
        u.krow = a.comp_row0 + (long long)u.unit * 2 * a.rows_comp;
        u.first_tile = 0;
        u.full = false;
    } else {
        const int x = w.f0 + (v - w.comp_tiles);
        u.unit = x / a.tiles_full;
        u.tile = x - u.unit * a.tiles_full;
        u.tiles = a.tiles_full;
        u.len = a.len_full;
        u.b = u.unit / a.n_full;
        u.head = a.head_of_slot[u.unit - u.b * a.n_full];
        u.rows = a.rows_full;
        u.krow = a.full_row0 + (long long)u.unit * 2 * a.rows_full;
        u.first_tile = u.unit * a.tiles_full;
        u.full = true;
    }
    return u;
}

// Launchers (defined in the .cu files).
cudaError_t launch_append(const AppendArgs& a, cudaStream_t stream);
cudaError_t launch_decode(const DecodeArgs& a, const CUtensorMap* tmap, int head_dim, int grid,
                          int stages, int groups, cudaStream_t stream);
cudaError_t prepare_decode_kernels(int head_dim);
size_t decode_smem_bytes(int head_dim, int stages, int group, int groups);

}  // namespace rlkv
