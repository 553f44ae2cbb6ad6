// Internal definitions shared by the host API and the kernels of librlkv.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace rlkv {

constexpr int kTile = 64;        // tokens per K/V tile (one pipeline stage holds a K and a V tile)
constexpr int kMaxGroup = 8;     // query heads per KV head handled by one tile pass
constexpr int kMaxKvHeads = 128; // KV heads per layer (their order travels in the kernel arguments)
constexpr int kMaxStepLayers = 128;  // layers whose appends rlkv_step does in one launch
constexpr int kMaxStepHeads = 4096;  // layers * kv_heads that one whole-step decode launch may serve
constexpr int kGroupWarps = 4;   // consumer warps that share one tile (16 tokens each)
constexpr int kMaxConsumerGroups = 3;
constexpr int kMaxDynamicSmem = 227 * 1024;
constexpr int kMergePad = 4;     // floats of padding per head row in the cross-warp merge area
constexpr int kEpilogueWarps = 2;  // warps that merge the consumer warps' states and the split partials
constexpr int kMergeBuffers = 2;   // hand-off buffers between consumer warps and epilogue warps
constexpr int kMaxRounds = 10;   // factoring rounds of the work schedule
constexpr int kItemRing = 4;     // work-item descriptors in flight between producer and consumers
constexpr int kTraceWords = 40;  // debug trace: 64-bit words per CTA
constexpr int kMaxTodo = 64;      // split merges a CTA may put off until its stream has ended
constexpr int kMaxPend = 16;      // partial segments of a CTA whose tickets are drawn when its stream has ended
constexpr int kMaxPagedBatch = 512;   // sequences one launch over the paged cache may serve
constexpr int kMaxSeqPages = 1024;    // 64-token pages one sequence may hold (65536 tokens)
constexpr int kClaimAhead = 3;   // the producer asks for its next work item this many tiles before the current one ends

// Kernel status codes (device error word).
enum : int {
    kStatusOk = 0,
    kStatusFullWaitTimeout = 1,   // a consumer gave up waiting for a tile to land
    kStatusEmptyWaitTimeout = 2,  // the producer gave up waiting for a stage to be released
    kStatusDrainTimeout = 3,      // the producer gave up waiting for its own copies in flight
    kStatusItemWaitTimeout = 4,   // a wait on the work-item ring ran out
    kStatusClaimWaitTimeout = 5,  // a wait between producer and claim warp ran out
    kStatusMergeWaitTimeout = 6,  // a wait between consumer warps and epilogue warps ran out
    kStatusSmemMisaligned = 7,    // dynamic shared memory does not start on a 1024-byte boundary
    kStatusPageWaitTimeout = 8    // the producer gave up waiting for page-table entries
};

// What a decode kernel is compiled for.
enum : int {
    kModePlain = 0,   // the lock-step cache: full and compressed heads, one length for the whole batch
    kModeMixed = 1,   // mixed attention (Eq. 1) over a lock-step cache whose heads are all full
    kModePaged = 2,   // the paged cache: one length per sequence, full heads in 64-token pages
    kModePagedFp8 = 3, // the paged cache with every K/V row (pages and rings) held as 8-bit E4M3 codes
    kModeStep = 4     // the lock-step cache, every layer of a decode step in one launch
};

// One record of split-KV partial results: running max and sum (log2 domain) of the G query heads
// of a unit, padded to a multiple of four floats, then their un-normalised output rows.
__host__ __device__ constexpr int partial_head_floats(int group) { return (2 * group + 3) / 4 * 4; }
__host__ __device__ constexpr int partial_floats(int head_dim, int group) {
    return partial_head_floats(group) + group * head_dim;
}

// ---- work decomposition -------------------------------------------------------------------------
// Units are (batch row, head-of-class): U FULL units of tf 64-row tiles each and Uc COMPRESSED
// units of tc tiles each (sink + ring rows).  Their tiles form one flat space of T tiles, laid out
// in BANDS: band 0 holds the first half of the tiles of every full unit (unit after unit), band 1
// half of what is left of every unit, and so on; the last band holds the rest of every full unit
// and, after them, the compressed units.  The space is cut into work items, contiguous tile
// ranges, by "factoring": band r < R is handed to the P CTAs in P equal items, so items shrink
// geometrically (few split points while everything is busy, fine grain at the end); the last band
// is cut into items of min_sz tiles.  CTA c starts with item c; later items are claimed from an
// atomic counter, so a CTA on a slow path to memory simply takes fewer of them.
// A SEGMENT is the part of one unit inside one item (a run of consecutive tiles of the unit).  A
// segment that is not the whole unit yields an (m, l, O) partial; the last CTA to deliver a
// partial of a unit merges them.  Because every unit has a slice in every band, every unit ends
// up with a similar, small number of partials.
// A launch with many more units than CTAs (a whole decode step in one launch) puts a PREFIX in front
// of the bands: the first U0 full units lie there whole, unit after unit, and are cut into P equal
// items (items 0 .. P-1, one per CTA), so most units are streamed in one piece by one CTA and only
// the units an item boundary falls into are split.  The remaining U - U0 units follow in bands as
// above (`rounds` = 0: in one band, i.e. unit after unit, cut into items of min_sz tiles).
// `unit_items`: the prefix is handed out unit by unit instead (one item per unit, CTA c starts with
// unit c and the others are claimed): for units of unequal real length (a paged batch of sequences of
// different lengths), where P equal tile ranges would not be P equal amounts of work.
struct Schedule {
    int P;                      // CTAs
    int R;                      // bands handed out in P equal items (the factoring rounds)
    int min_sz;                 // tiles per item in the last band
    int n_items;
    int n_slots;                // partial records the launch may write
    int U, tf, Uc, tc;
    int T;                      // tiles in the flat space
    int U0;                     // full units in the whole-unit prefix (0: no prefix)
    int x0, k0, s0;             // first flat tile, first item and first partial record after the prefix
    int pq, prem;               // the prefix's P items have pq tiles, the first prem one more
    int kc;                     // first item that holds compressed tiles only (n_items if there is none)
    int base[kMaxRounds + 2];   // first flat tile of band r <= R; base[R+1]: first compressed tile
    int tb[kMaxRounds + 2];     // first tile, inside a full unit, of its slice in band r; tb[R+1] = tf
    int slot0[kMaxRounds + 1];  // first partial record of band r
    int iq[kMaxRounds];         // band r < R: its P items have iq[r] tiles, the first irem[r] one more
    int irem[kMaxRounds];
};

inline Schedule make_schedule(int U, int tf, int Uc, int tc, int P, int min_sz, int U0 = 0, int rounds = kMaxRounds,
                              bool unit_items = false)
{
    Schedule s{};
    s.P = P;
    s.min_sz = min_sz;
    s.U = U;
    s.tf = U > 0 ? tf : 0;
    s.Uc = Uc;
    s.tc = Uc > 0 ? tc : 0;
    if (U0 > U) U0 = U;
    if (U0 < 0 || (long long)U0 * s.tf < P) U0 = 0;  // every prefix item holds at least one tile
    s.U0 = U0;
    s.x0 = U0 * s.tf;
    if (unit_items && U0 < P) U0 = s.U0 = s.x0 = 0;          // every CTA starts with a unit of its own
    s.k0 = U0 > 0 ? (unit_items ? U0 : P) : 0;
    s.s0 = U0 > 0 ? s.k0 + U0 : 0;
    s.pq = U0 > 0 ? (unit_items ? s.tf : s.x0 / P) : 0;
    s.prem = U0 > 0 && !unit_items ? s.x0 % P : 0;
    const int Ub = U - U0;  // full units laid out in bands
    int r = 0;
    s.base[0] = s.x0;
    s.tb[0] = 0;
    while (r < rounds && r < kMaxRounds) {
        const int bw = (s.tf - s.tb[r]) / 2;
        if ((long long)Ub * bw / P < 2 * min_sz) break;
        s.tb[r + 1] = s.tb[r] + bw;
        s.base[r + 1] = s.base[r] + Ub * bw;
        s.slot0[r] = s.s0 + r * (P + Ub);
        s.iq[r] = Ub * bw / P;
        s.irem[r] = Ub * bw % P;
        ++r;
    }
    s.R = r;
    s.slot0[r] = s.s0 + r * (P + Ub);
    s.tb[r + 1] = s.tf;
    s.base[r + 1] = s.base[r] + Ub * (s.tf - s.tb[r]);
    s.T = s.base[r + 1] + s.Uc * s.tc;
    const int n_final = (s.T - s.base[r] + min_sz - 1) / min_sz;
    s.n_items = s.k0 + r * P + n_final;
    s.n_slots = s.slot0[r] + n_final + Ub + Uc;
    // the last band's items are min_sz tiles from base[r] on: the first one that starts among the compressed tiles
    s.kc = s.Uc > 0 ? s.k0 + r * P + (s.base[r + 1] - s.base[r] + min_sz - 1) / min_sz : s.n_items;
    if (s.kc > s.n_items) s.kc = s.n_items;
    return s;
}

// The order in which items are handed out.  CTA c starts with item c (c < P); the i-th claim after that
// (k = P + i) gets the items that hold compressed units first and the others, in order, after them: an
// item of compressed units is many short segments, each with its own query fetch and hand-off, and
// takes longer than its tiles say -- such items must not be the last ones of the launch.  Which CTA
// processes which item never changes a result.
__host__ __device__ inline int claim_to_item(const Schedule& s, int k)
{
    if (k < s.P || k >= s.n_items) return k;
    const int first = s.kc > s.P ? s.kc : s.P;  // first claimable item of compressed units
    const int nc = s.n_items - first, j = k - s.P;
    return j < nc ? first + j : s.P + (j - nc);
}

// Upper bound of n_slots over every tf' <= tf with everything else the same (no prefix).
inline long long max_slots(int U, int tf, int Uc, int tc, int P, int min_sz)
{
    const Schedule s = make_schedule(U, tf, Uc, tc, P, min_sz);
    // tiles of the last band: under 4*min_sz*P + 2U unless the rounds ran out first
    const long long by_size = 4ll * min_sz * P + 2ll * U;
    const long long by_rounds = (long long)U * ((tf >> kMaxRounds) + 2);
    const long long last = (by_size > by_rounds ? by_size : by_rounds) + (long long)Uc * tc;
    return (long long)s.R * (P + U) + last / min_sz + U + Uc + 4;
}

// First tile of item k (k >= n_items gives T).
__host__ __device__ inline int item_start(const Schedule& s, int k)
{
    if (k >= s.n_items) return s.T;
    if (k < s.k0) return k * s.pq + (k < s.prem ? k : s.prem);
    k -= s.k0;
    const int rp = s.R * s.P;
    if (k < rp) {
        const int r = k / s.P, j = k - r * s.P;
        return s.base[r] + j * s.iq[r] + (j < s.irem[r] ? j : s.irem[r]);
    }
    return s.base[s.R] + (k - rp) * s.min_sz;
}

// The item that holds flat tile x.
__host__ __device__ inline int item_of_tile(const Schedule& s, int x)
{
    if (x < s.x0) {
        const int big = s.prem * (s.pq + 1);
        return x < big ? x / (s.pq + 1) : s.prem + (x - big) / s.pq;
    }
    for (int r = 0; r < s.R; ++r)
        if (x < s.base[r + 1]) {
            const int y = x - s.base[r], big = s.irem[r] * (s.iq[r] + 1);
            return s.k0 + r * s.P + (y < big ? y / (s.iq[r] + 1) : s.irem[r] + (y - big) / s.iq[r]);
        }
    return s.k0 + s.R * s.P + (x - s.base[s.R]) / s.min_sz;
}

// Where flat tile x lies: the unit (index over both classes, full units first), the tile inside
// the unit, how many tiles of the unit follow consecutively in the flat space from x on (x
// included), and the band (-1: the whole-unit prefix).
struct TilePos {
    int uid, tile, run, band;
};
__host__ __device__ inline TilePos tile_pos(const Schedule& s, int x)
{
    TilePos p;
    if (x < s.x0) {
        p.uid = x / s.tf;
        p.tile = x - p.uid * s.tf;
        p.run = s.tf - p.tile;
        p.band = -1;
    } else if (x < s.base[s.R + 1]) {
        int r = s.R;
        for (int i = 0; i < s.R; ++i)
            if (x < s.base[i + 1]) {
                r = i;
                break;
            }
        const int bw = s.tb[r + 1] - s.tb[r], y = x - s.base[r];
        const int unit = y / bw, off = y - unit * bw;
        p.uid = s.U0 + unit;
        p.tile = s.tb[r] + off;
        p.run = bw - off;
        p.band = r;
    } else {
        const int y = x - s.base[s.R + 1];
        const int unit = y / s.tc, off = y - unit * s.tc;
        p.uid = s.U + unit;
        p.tile = off;
        p.run = s.tc - off;
        p.band = s.R;
    }
    return p;
}

// The partial record of the segment of unit `uid` inside item `item` of band `band`: along a band
// (and along the prefix) every new segment raises the item index or the unit index, so their sum
// numbers the segments.
__host__ __device__ inline int partial_slot(const Schedule& s, int band, int item, int uid)
{
    if (band < 0) return item + uid;
    return s.slot0[band] + (item - s.k0 - band * s.P) + (uid - s.U0);
}

// The partial records of unit `uid` in band `band` >= 0: first record and how many (0 if the unit
// has no slice there).  Full units outside the prefix have a slice in every band, compressed units
// only in the last; a unit of the prefix reports its records under band 0 and none elsewhere.
// `tiles`: how many of the unit's tiles exist (paged cache: a sequence shorter than the longest one
// of the call); segments that hold none of them deliver no record.
__host__ __device__ inline void unit_partials(const Schedule& s, int uid, int band, int& slot, int& count,
                                              int tiles = 0x7fffffff)
{
    int first, width;
    const bool prefix = uid < s.U0;
    if (prefix) {
        width = band == 0 ? (s.tf < tiles ? s.tf : tiles) : 0;
        first = uid * s.tf;
    } else if (uid < s.U) {
        width = s.tb[band + 1] - s.tb[band];
        first = s.base[band] + (uid - s.U0) * width;
        if (width > tiles - s.tb[band]) width = tiles - s.tb[band];
    } else {
        width = band == s.R ? (s.tc < tiles ? s.tc : tiles) : 0;
        first = s.base[s.R + 1] + (uid - s.U) * s.tc;
    }
    if (width <= 0) {
        slot = 0;
        count = 0;
        return;
    }
    const int kf = item_of_tile(s, first), kl = item_of_tile(s, first + width - 1);
    slot = partial_slot(s, prefix ? -1 : band, kf, uid);
    count = kl - kf + 1;
}

// Everything a decode launch needs about one layer.  Passed by value.
struct DecodeArgs {
    const __nv_bfloat16* pool;  // base of the row pool, rows of head_dim bf16
    long long full_row0;        // first pool row of the layer's full-head region
    long long comp_row0;        // first pool row of the layer's compressed-head region
    const __nv_bfloat16* q;     // [batch][q_heads][head_dim]
    float* out;                 // [batch][q_heads][head_dim]; bf16 elements instead of fp32 if out_bf16
    float* partials;            // [sched.n_slots][partial_floats]
    int* tickets;               // one per unit of this layer, zero between launches
    unsigned int* claim_counter;  // items claimed beyond the first P, over all launches so far (never reset)
    unsigned int claim_base;      // its value when this launch starts: every launch adds exactly sched.n_items
    int dep_wait;               // how the launch is ordered against its predecessor in the stream (see the
                                // first lines of decode_kernel and step_launch_mode): 0 ordinary, 1 it may run
                                // beside the step's append launch, 2 it may run beside the decode launch before it
    int* status;                // device error word
    unsigned long long* trace;  // debug: [grid][kTraceWords]
    int n_full, n_comp;         // heads of each class in this layer
    int rows_full, rows_comp;   // allocated rows per head (multiples of kTile)
    int len_full, len_comp;     // valid rows per head right now: n and min(n, sink+window)
    int batch, group, q_heads;
    float scale_log2;           // log2(e) / sqrt(head_dim)
    int trace_on;
    int out_bf16;               // results are rounded to bf16 (nearest even) when they are stored
    // Mixed attention (paper, Eq. 1; MIXED kernels only).  Every head of the layer is full and holds
    // more than sink + window tokens.  The first class of units covers, per (batch row, head), the
    // len_full rows between the sink and the window (from row local_sink on); the second class holds a
    // LOCAL unit over the sink and the window: tiles 0 .. local_sink_tiles-1 cover rows
    // [0, local_sink), the tiles after them rows [local_win0, local_win0 + local_win_len).  No row
    // belongs to both; the local branch of Eq. 1 is the merge of the local unit's partial records, the
    // full branch the merge of both units' (merge_units).
    // A launch that also appends the step's token (lock-step cache, one layer): the caller's new rows,
    // [batch][kv_heads][head_dim]; token len_full - 1 of every head is written by the CTA that reads the
    // tile it belongs to (row len_full - 1 of a full head, the ring slot of a compressed head).  Null otherwise.
    const __nv_bfloat16* new_k;
    const __nv_bfloat16* new_v;
    int new_sink, new_window;
    const float* alpha;         // gates of the layer's KV heads (device, [kv_heads]); null otherwise
    int local_sink, local_sink_tiles, local_win0, local_win_len;
    Schedule sched;
    unsigned char head_of_slot[kMaxKvHeads];  // KV head of full slot 0..n_full-1, then of the compressed slots
};

// A whole decode step in one launch (kModeStep kernels): what DecodeArgs cannot say.  Every layer holds
// the same number of tokens.  The full units of all layers form one list, layer after layer (inside a
// layer: batch row, then full-head slot), and so do the compressed units; q and out are the step's
// [layers][batch][q_heads][head_dim] arrays, so "batch row" l * batch + b addresses them directly.
struct StepArgs {
    const int* head_of_slot;            // device, int [n_layers][kv_heads]: KV head of each slot (full slots first)
    int n_layers, kv_heads, batch;
    int full_base[kMaxStepLayers + 1];  // first full unit of layer l = batch * (full heads of the layers before it)
    int comp_base[kMaxStepLayers + 1];  // first compressed unit of layer l, counted from the first compressed unit
    int full_row0[kMaxStepLayers];      // first pool row of the layer's full-head / compressed-head region
    int comp_row0[kMaxStepLayers];
};

// Paged cache (kModePaged kernels): what DecodeArgs cannot say.  The launch serves `batch` sequences;
// entry b of q and out belongs to request slot seq_slot[b], which holds seq_len[b] tokens in this
// layer.  Units are laid out as for the lock-step cache with every full unit given the tiles of the
// LONGEST sequence; a unit's tiles past its own length are skipped by producer and consumers alike.
// Full heads: token t of slot s lives in page page_table[s * table_stride + t / 64], row t % 64; page
// p of full-head slot f of the layer starts at pool row full_row0 + ((f * n_pages + p) * 2) * 64 (K
// rows, then the 64 V rows).  Compressed heads: the ring of request slot s and compressed-head slot
// c starts at pool row comp_row0 + ((s * n_comp + c) * 2) * rows_comp.
struct PagedArgs {
    const int* page_table;
    int table_stride;  // entries per request slot, a multiple of 4
    int n_pages;       // physical pages per full head
    int cap;           // sink + window
    // 8-bit pages (kModePagedFp8): a page is 16 KB, K codes [64 tokens][128] then V codes TRANSPOSED
    // [128][64 tokens]; page p of full-head slot f of the layer is page page0_8 + f * n_pages + p of the
    // 8-bit pool; the ring of request slot s and compressed-head slot c is the ring_tiles pages from
    // ring0_8 + (s * n_comp + c) * ring_tiles on (ring row r in page r / 64, row r % 64).
    // x_hat = value(code) * scale with one scale per KV head (indexed by head) for K, V.
    int page0_8, ring0_8, ring_tiles;
    float k_scale[kMaxKvHeads], v_scale[kMaxKvHeads];
    int seq_len[kMaxPagedBatch];
    unsigned short seq_slot[kMaxPagedBatch];
    // A whole step in one launch (step.n_layers > 1; every listed sequence holds the same number of tokens
    // in all layers): the units of all layers form one list as for the lock-step cache (StepArgs, with
    // `batch` = sequences of the call), q and out are [layers][batch][q_heads][head_dim], and what the
    // fields above and DecodeArgs say per layer comes per layer: the regions' first pool rows from
    // `step`, the first 8-bit pages from these arrays, the scales from device memory (k_scale
    // [layers][kv_heads], then v_scale).  step.n_layers <= 1: a launch for one layer, these are unused.
    StepArgs step;
    const float* scales;
    int page0_8_of[kMaxStepLayers], ring0_8_of[kMaxStepLayers];
};
// The tensor map over the 8-bit pool: rows of 128 bytes, boxes of 128 rows = one page (64 rows of K
// codes, then the transposed V codes, two d per row).
struct alignas(64) PagedFp8Args {
    PagedArgs pa;
    alignas(64) CUtensorMap map_k;
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
    int overlap;                // the launch may start before the kernel before it has completed: wait for it first
};

// What producer and consumers need to know about the unit behind a flat tile.
struct UnitInfo {
    TilePos pos;
    int tiles;       // tiles of the unit
    int len;         // valid rows of the unit
    int b, head;     // batch row (whole-step launch of the lock-step cache: layer * batch + batch row), KV head
    int qrow;        // the unit's G query (and output) rows start at row qrow * q_heads + head * G
    int row0;        // lock-step cache: first pool row of the unit's K rows; its V rows start `vrows` further on
    int vrows;
    int layer;       // the layer (0 in a launch for one layer), the unit's slot among the heads of its class in
    int slot;        // that layer, and how many heads of that class the layer has
    int nclass;
};

// The layer a unit of a whole-step launch belongs to: the last l with base[l] <= unit.
__device__ inline int step_layer(const int* base, int n_layers, int unit)
{
    int lo = 0, hi = n_layers - 1;
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (base[mid] <= unit) lo = mid;
        else hi = mid - 1;
    }
    return lo;
}

// `st`, `heads`: whole-step launches only -- the layer tables and the KV head of every slot
// ([layer][kv_heads] bytes), both in shared memory.
template <int MODE = kModePlain>
__device__ inline UnitInfo locate(const DecodeArgs& a, int x, const PagedArgs* pg = nullptr, const StepArgs* st = nullptr,
                                  const unsigned char* heads = nullptr)
{
    constexpr bool MIXED = MODE == kModeMixed;
    UnitInfo u;
    u.pos = tile_pos(a.sched, x);
    u.row0 = 0;
    u.vrows = 0;
    u.layer = 0;
    u.slot = 0;
    u.nclass = 0;
    if ((MODE == kModePaged || MODE == kModePagedFp8) && pg->step.n_layers > 1) {  // the paged cache, a whole step
        const StepArgs* ps = &pg->step;
        const bool full = u.pos.uid < a.sched.U;
        const int unit = full ? u.pos.uid : u.pos.uid - a.sched.U;
        const int* base = full ? ps->full_base : ps->comp_base;
        const int l = step_layer(base, ps->n_layers, unit);
        const int local = unit - base[l];
        const int nf = (ps->full_base[l + 1] - ps->full_base[l]) / ps->batch;
        u.nclass = full ? nf : ps->kv_heads - nf;
        u.b = local / u.nclass;
        u.slot = local - u.b * u.nclass;
        u.layer = l;
        u.qrow = l * ps->batch + u.b;
        u.tiles = full ? a.sched.tf : a.sched.tc;
        u.head = heads[l * ps->kv_heads + (full ? u.slot : nf + u.slot)];
        const int n = pg->seq_len[u.b];
        u.len = full ? n : (n < pg->cap ? n : pg->cap);
        return u;
    }
    if (MODE == kModeStep) {
        const bool full = u.pos.uid < a.sched.U;
        const int unit = full ? u.pos.uid : u.pos.uid - a.sched.U;
        const int* base = full ? st->full_base : st->comp_base;
        const int l = step_layer(base, st->n_layers, unit);
        const int local = unit - base[l];
        const int nf = (st->full_base[l + 1] - st->full_base[l]) / st->batch;
        const int per_row = full ? nf : st->kv_heads - nf;  // units of this class per batch row of the layer
        const int b = local / per_row, slot = local - b * per_row;
        u.layer = l;
        u.slot = slot;
        u.nclass = per_row;
        u.tiles = full ? a.sched.tf : a.sched.tc;
        u.len = full ? a.len_full : a.len_comp;
        u.b = l * st->batch + b;
        u.qrow = u.b;
        u.head = heads[l * st->kv_heads + (full ? slot : nf + slot)];
        u.vrows = full ? a.rows_full : a.rows_comp;
        u.row0 = (full ? st->full_row0[l] : st->comp_row0[l]) + local * 2 * u.vrows;
        return u;
    }
    if (u.pos.uid < a.sched.U) {
        u.tiles = a.sched.tf;
        u.len = a.len_full;
        u.b = u.pos.uid / a.n_full;
        u.slot = u.pos.uid - u.b * a.n_full;
        u.nclass = a.n_full;
        u.head = a.head_of_slot[u.slot];
        u.vrows = a.rows_full;
        u.row0 = (int)(a.full_row0 + (long long)u.pos.uid * 2 * a.rows_full);
        // mixed attention: the first class covers the tokens between the sink and the window only (len_full
        // of them, from row local_sink on); sink and window are read once, by the local unit
        if (MIXED) u.row0 += a.local_sink;
    } else if (MIXED) {  // the local unit of full unit uid - U
        const int unit = u.pos.uid - a.sched.U;
        u.tiles = a.sched.tc;
        u.len = 0;       // its tiles' rows come from local_tile
        u.b = unit / a.n_full;
        u.slot = unit - u.b * a.n_full;
        u.nclass = a.n_full;
        u.head = a.head_of_slot[u.slot];
        u.vrows = a.rows_full;
        u.row0 = (int)(a.full_row0 + (long long)unit * 2 * a.rows_full);
    } else {
        const int unit = u.pos.uid - a.sched.U;
        u.tiles = a.sched.tc;
        u.len = a.len_comp;
        u.b = unit / a.n_comp;
        u.slot = unit - u.b * a.n_comp;
        u.nclass = a.n_comp;
        u.head = a.head_of_slot[a.n_full + u.slot];
        u.vrows = a.rows_comp;
        u.row0 = (int)(a.comp_row0 + (long long)unit * 2 * a.rows_comp);
    }
    u.qrow = u.b;
    if (MODE == kModePaged || MODE == kModePagedFp8) {  // this sequence's own length
        const int n = pg->seq_len[u.b];
        const bool full = u.pos.uid < a.sched.U;
        u.len = full ? n : (n < pg->cap ? n : pg->cap);
        u.nclass = full ? a.n_full : a.n_comp;
        u.slot = full ? u.pos.uid - u.b * a.n_full : u.pos.uid - a.sched.U - u.b * a.n_comp;
    }
    return u;
}

// The unit after `u` in the flat tile space, for the producer's walk along an item: inside one region
// (the whole-unit prefix, a band, the compressed units) the slices of consecutive units of a class
// follow one another, so the next segment's unit is u's successor and nothing has to be looked up
// from scratch (locate costs four divisions and a binary search; a compressed unit is two tiles
// long).  `u` must come from locate or from this function; tile, run and band of the new position are
// the caller's (they are the region's).  Returns false where the successor lies in the next layer of a
// whole-step launch: the caller then calls locate.
template <int MODE>
__device__ inline bool next_unit(const DecodeArgs& a, UnitInfo& u, const PagedArgs* pg, const StepArgs* st,
                                 const unsigned char* heads)
{
    // (mixed attention: a local unit is addressed like the full unit of the same head)
    const bool full = u.pos.uid < a.sched.U || MODE == kModeMixed;
    if (MODE == kModePaged || MODE == kModePagedFp8) {  // u.b: the sequence of the call; rows come from pages
        const bool whole = pg->step.n_layers > 1;
        ++u.pos.uid;
        if (++u.slot == u.nclass) {
            u.slot = 0;
            ++u.b;
            if (whole && u.b == pg->step.batch) return false;  // the layer's last sequence is done
            const int n = pg->seq_len[u.b];
            u.len = full ? n : (n < pg->cap ? n : pg->cap);
        }
        u.qrow = whole ? u.layer * pg->step.batch + u.b : u.b;
        if (whole) u.head = heads[u.layer * pg->step.kv_heads + (full ? u.slot : pg->step.kv_heads - u.nclass + u.slot)];
        else u.head = a.head_of_slot[(full ? 0 : a.n_full) + u.slot];
        return true;
    }
    ++u.pos.uid;
    u.row0 += 2 * u.vrows;  // the units of a class lie one after the other in a layer's region of the pool
    if (++u.slot == u.nclass) {
        u.slot = 0;
        ++u.b;
        if (MODE == kModeStep && u.b == (u.layer + 1) * st->batch) return false;  // the layer's last batch row is done
    }
    u.qrow = u.b;
    if (MODE == kModeStep) u.head = heads[u.layer * st->kv_heads + (full ? u.slot : st->kv_heads - u.nclass + u.slot)];
    else u.head = a.head_of_slot[(full ? 0 : a.n_full) + u.slot];
    return true;
}

// Paged cache: how many tiles of unit `uid` exist.
__device__ inline int paged_unit_tiles(const DecodeArgs& a, const PagedArgs* pg, int uid)
{
    const bool full = uid < a.sched.U;
    int b;
    if (pg->step.n_layers > 1) {
        const StepArgs* ps = &pg->step;
        const int unit = full ? uid : uid - a.sched.U;
        const int* base = full ? ps->full_base : ps->comp_base;
        const int l = step_layer(base, ps->n_layers, unit);
        const int nf = (ps->full_base[l + 1] - ps->full_base[l]) / ps->batch;
        b = (unit - base[l]) / (full ? nf : ps->kv_heads - nf);
    } else {
        b = full ? uid / a.n_full : (uid - a.sched.U) / a.n_comp;
    }
    int n = pg->seq_len[b];
    if (!full && n > pg->cap) n = pg->cap;
    return (n + kTile - 1) / kTile;
}

// Mixed attention: tile `tile` of a local unit holds rows [row, row + valid) of its head; what
// follows them in the 64-row box is fetched and masked.
__device__ inline void local_tile(const DecodeArgs& a, int tile, int& row, int& valid)
{
    if (tile < a.local_sink_tiles) {
        row = tile * kTile;
        valid = a.local_sink - row;
    } else {
        const int off = (tile - a.local_sink_tiles) * kTile;
        row = a.local_win0 + off;
        valid = a.local_win_len - off;
    }
    if (valid > kTile) valid = kTile;
}

#ifdef __CUDACC__
// Programmatic dependent launch: let the next kernel of the stream start / wait until the kernels
// before this one have completed and their writes are visible (no-ops for ordinary launches).
__device__ __forceinline__ void grid_dep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void grid_dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
#endif

// Launchers (defined in the .cu files).
// `overlap` (launch_decode): launch with programmatic stream serialization, so that the kernel may
// start while the kernel before it in the stream is still running.  Only for the decode launches of
// one step, whose inputs are complete before the step's first launch: consecutive layers use
// different copies of the scratch memory and touch nothing of each other; DecodeArgs::dep_wait says
// what the kernel waits for on the device.
cudaError_t launch_append(const AppendArgs& a, cudaStream_t stream);

// The appends of one token to every layer, in one launch (rlkv_step).
struct LayerDesc {
    long long full_row0, comp_row0;  // first pool row of the layer's full-head / compressed-head region
    int n_full, n_comp;
    long long page0_8, ring0_8;      // paged cache with 8-bit pages: the layer's first full-head page and first
                                     // ring page in the 8-bit pool
};
struct AppendAllArgs {
    __nv_bfloat16* pool;
    const LayerDesc* layers;    // device, [n_layers]
    const int* slot_of_head;    // device, [n_layers][kv_heads]
    const __nv_bfloat16* k;     // [n_layers][batch][kv_heads][head_dim]
    const __nv_bfloat16* v;
    int n_layers, rows_full, rows_comp, batch, kv_heads, head_dim, sink, window;
    int t0[kMaxStepLayers];     // token index appended to each layer
};
cudaError_t launch_append_all(const AppendAllArgs& a, cudaStream_t stream);
cudaError_t launch_decode(const DecodeArgs& a, const CUtensorMap* tmap, int head_dim, int grid,
                          int stages, int groups, cudaStream_t stream, bool overlap, int mode = kModePlain,
                          const PagedArgs* paged = nullptr, const PagedFp8Args* paged8 = nullptr,
                          const StepArgs* step = nullptr);
cudaError_t prepare_decode_kernels(int head_dim);
size_t decode_smem_bytes(int head_dim, int stages, int group, int groups, int mode = kModePlain);

// Paged cache: one token for each of n sequences of one layer / n_tokens tokens of one sequence.
// Entry i of k, v ([n][kv_heads][head_dim]) is token t[i] of request slot slot[i] (append) or token
// t0 + i of request slot slot[0] (prefill); page[j] is the physical page of page index
// first_page + j of the sequence (append: j = i, the page of token t[i]).  The kernel also records
// the pages in the device page table.
// With n_layers > 1 (rlkv_paged_step) the launch appends the same token positions to every layer: k, v
// are [n_layers][n][kv_heads][head_dim], slot_of_head is the table of layer 0 of [n_layers][kv_heads],
// and each layer's regions come from `layers`.
constexpr int kMaxAppendPages = 512;
struct PagedAppendArgs {
    __nv_bfloat16* pool;
    int* page_table;
    long long full_row0, comp_row0;
    const int* slot_of_head;    // [kv_heads]: >= 0 full slot, < 0: -(comp slot + 1)
    const __nv_bfloat16* k;
    const __nv_bfloat16* v;
    int n_full, n_comp, rows_comp, n_pages, table_stride;
    int kv_heads, head_dim, sink, window;
    int prefill;                // 0: n sequences, one token each; 1: one sequence, n tokens from t0
    int n, t0, first_page;
    int n_layers;               // 1 unless the launch serves every layer
    const LayerDesc* layers;    // device, [n_layers]; unused when n_layers == 1
    long long entry_stride;     // elements from one entry of k, v to the next (kv_heads * head_dim when contiguous)
    // 8-bit storage (null: 16-bit rows): the pool of pages and rings, 1 / scale per head of the first layer
    // served ([n_layers][kv_heads]), the layer's first page when n_layers == 1
    unsigned char* pool8;
    const float* k_inv;
    const float* v_inv;
    long long page0_8, ring0_8;
    int ring_tiles;             // pages per ring
    int page[kMaxAppendPages];
    int t[kMaxPagedBatch];
    unsigned short slot[kMaxPagedBatch];
};
cudaError_t launch_paged_append(const PagedAppendArgs& a, cudaStream_t stream);

}  // namespace rlkv
