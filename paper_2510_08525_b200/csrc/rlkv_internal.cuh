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
constexpr int kEpilogueWarps = 2;  // warps that merge the consumer warps' states and the split partials
constexpr int kMergeBuffers = 2;   // hand-off buffers between consumer warps and epilogue warps
constexpr int kMaxRounds = 10;   // factoring rounds of the work schedule
constexpr int kItemRing = 4;     // work-item descriptors in flight between producer and consumers
constexpr int kTraceWords = 8;   // debug trace: 64-bit words per CTA

// Kernel status codes (device error word).
enum : int {
    kStatusOk = 0,
    kStatusFullWaitTimeout = 1,   // a consumer gave up waiting for a tile to land
    kStatusEmptyWaitTimeout = 2,  // the producer gave up waiting for a stage to be released
    kStatusDrainTimeout = 3,      // the producer gave up waiting for its own copies in flight
    kStatusItemWaitTimeout = 4,   // a wait on the work-item ring ran out
    kStatusClaimWaitTimeout = 5,  // a wait between producer and claim warp ran out
    kStatusMergeWaitTimeout = 6,  // a wait between consumer warps and epilogue warps ran out
    kStatusSmemMisaligned = 7     // dynamic shared memory does not start on a 1024-byte boundary
};

// One record of split-KV partial results: running max and sum (log2 domain) of the G query heads
// of a unit, padded to a multiple of four floats, then their un-normalised output rows.
__host__ __device__ constexpr int partial_head_floats(int group) { return (2 * group + 3) / 4 * 4; }
__host__ __device__ constexpr int partial_floats(int head_dim, int group) {
    return partial_head_floats(group) + group * head_dim;
}

// ---- work decomposition -------------------------------------------------------------------------
// Units are (batch row, head-of-class).  The 64-row tiles of all units form one flat space of T
// tiles: the FULL units first (unit u owns tiles [u*tiles_full, (u+1)*tiles_full)), then the
// COMPRESSED units (tiles_comp tiles each: sink + ring rows).  The flat space is cut into work
// items, contiguous tile ranges, by "factoring": round r hands half of what is left to the P CTAs
// in P equal items, so items shrink geometrically (few split points while everything is busy,
// fine grain at the end); once an item would fall under 2*min_sz tiles the rest is cut into items
// of min_sz tiles.  CTA c starts with item c; later items are claimed from an atomic counter, so a
// CTA on a slow path to memory simply takes fewer of them.  An item may begin and end inside a
// unit: such a segment yields an (m, l, O) partial and the last CTA to deliver a partial of a unit
// merges them.
struct Schedule {
    int T;                      // tiles in the flat space
    int P;                      // CTAs
    int R;                      // factoring rounds
    int min_sz;                 // tiles per item in the final section
    int n_items;
    int base[kMaxRounds + 1];   // first tile of round r; base[R] = first tile of the final section
    int len[kMaxRounds];        // tiles handed out in round r
};

inline Schedule make_schedule(int T, int P, int min_sz)
{
    Schedule s{};
    s.T = T;
    s.P = P;
    s.min_sz = min_sz;
    int r = 0;
    s.base[0] = 0;
    while (r < kMaxRounds) {
        const int rem = T - s.base[r];
        const int len = rem / 2;
        if (len / P < 2 * min_sz) break;
        s.len[r] = len;
        s.base[r + 1] = s.base[r] + len;
        ++r;
    }
    s.R = r;
    const int rem = T - s.base[r];
    s.n_items = r * P + (rem + min_sz - 1) / min_sz;
    return s;
}

// Upper bound of n_items over every T' <= T with the same P and min_sz.
inline int max_items(int T, int P, int min_sz)
{
    const Schedule s = make_schedule(T, P, min_sz);
    // the final section holds fewer than 4*min_sz*P + 2 tiles unless the rounds ran out first
    const int by_size = 4 * P + 2, by_rounds = (T >> kMaxRounds) / min_sz + 2;
    return (s.R + 1) * P + (by_size > by_rounds ? by_size : by_rounds);
}

// First tile of item k (k >= n_items gives T).
__host__ __device__ inline int item_start(const Schedule& s, int k)
{
    if (k >= s.n_items) return s.T;
    const int rp = s.R * s.P;
    if (k < rp) {
        const int r = k / s.P, j = k - r * s.P;
        return s.base[r] + (int)(((long long)j * s.len[r]) / s.P);
    }
    return s.base[s.R] + (k - rp) * s.min_sz;
}

// The item that holds flat tile x.
__host__ __device__ inline int item_of_tile(const Schedule& s, int x)
{
    for (int r = 0; r < s.R; ++r)
        if (x < s.base[r + 1])
            return r * s.P + (int)((((long long)(x - s.base[r]) + 1) * s.P - 1) / s.len[r]);
    return s.R * s.P + (x - s.base[s.R]) / s.min_sz;
}

// Everything a decode launch needs about one layer.  Passed by value.
struct DecodeArgs {
    const __nv_bfloat16* pool;  // base of the row pool, rows of head_dim bf16
    long long full_row0;        // first pool row of the layer's full-head region
    long long comp_row0;        // first pool row of the layer's compressed-head region
    const int* head_of_slot;    // [kv_heads]: KV head of full slot 0..n_full-1, then of comp slots
    const __nv_bfloat16* q;     // [batch][q_heads][head_dim]
    float* out;                 // [batch][q_heads][head_dim]
    float* partials;            // [2 slots][part_items][partial_floats]
    long long part_items;       // items the partial area is laid out for (>= sched.n_items)
    int* tickets;               // one per unit of this layer, zero between launches
    int* counters;              // [0] items claimed beyond the first P, [1] CTAs finished; zero between launches
    int* status;                // device error word
    unsigned long long* trace;  // debug: [grid][kTraceWords]
    int n_full, n_comp;         // heads of each class in this layer
    int rows_full, rows_comp;   // allocated rows per head (multiples of kTile)
    int len_full, len_comp;     // valid rows per head right now: n and min(n, sink+window)
    int batch, group, q_heads;
    int tiles_full, tiles_comp; // ceil(len / kTile) per head of each class
    int full_tiles;             // batch*n_full*tiles_full: where the compressed units start
    int full_units;             // batch*n_full
    float scale_log2;           // log2(e) / sqrt(head_dim)
    int trace_on;
    Schedule sched;
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

struct UnitInfo {
    int uid;         // unit index over both classes (full units first): the ticket index
    int tile;        // tile index inside the unit
    int tiles;       // tiles of the unit
    int len;         // valid rows of the unit
    int b, head;     // batch row, KV head
    int first_tile;  // flat index of the unit's tile 0
};

// The unit and tile behind flat tile x.
__device__ inline UnitInfo locate(const DecodeArgs& a, int x)
{
    UnitInfo u;
    if (x < a.full_tiles) {
        const int unit = x / a.tiles_full;
        u.uid = unit;
        u.tile = x - unit * a.tiles_full;
        u.tiles = a.tiles_full;
        u.len = a.len_full;
        u.b = unit / a.n_full;
        u.head = a.head_of_slot[unit - u.b * a.n_full];
        u.first_tile = unit * a.tiles_full;
    } else {
        const int y = x - a.full_tiles;
        const int unit = y / a.tiles_comp;
        u.uid = a.full_units + unit;
        u.tile = y - unit * a.tiles_comp;
        u.tiles = a.tiles_comp;
        u.len = a.len_comp;
        u.b = unit / a.n_comp;
        u.head = a.head_of_slot[a.n_full + (unit - u.b * a.n_comp)];
        u.first_tile = a.full_tiles + unit * a.tiles_comp;
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
