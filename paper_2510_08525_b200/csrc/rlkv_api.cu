// Host side of librlkv: argument checks, the two-class cache layout, launches.
//
// Device buffer layout (all sections 1024-byte aligned):
//   pool      rows of head_dim bf16.  Per layer: the full-head region
//             [batch][n_full(layer)][K|V][rows_full][D], then the compressed-head region
//             [batch][n_comp(layer)][K|V][rows_comp][D].  rows_full = max_len and
//             rows_comp = sink+window, each rounded up to the 64-row tile, so a tile never reaches
//             into a neighbouring head and a compressed head owns a constant number of rows
//             (the constant-size pool of Section 4.3 of the paper).
//   tables    int32 slot_of_head[layers][kv_heads], head_of_slot[layers][kv_heads]
//   tickets   int32 [layers][2*batch*kv_heads] (split bookkeeping, zero between launches; one per unit of a
//             launch -- a whole-step launch numbers the units of all its layers in one list)
//   tables    then LayerDesc[layers] (where each layer's regions start; for the step's append launch)
//   status    int32 kernel status word, then two work-claim counters (they only grow; consecutive
//             launches of a step alternate between them)
//   partials  float [2][max_slots][partial_floats]  (split-KV scratch; the two halves alternate too)
//   staging   k, v, q (twice: calls alternate) and out of one whole step, for rlkv_step_host
//   trace     uint64 [max_grid][40]  (debug trace of the decode kernel)
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <atomic>
#include <new>
#include <vector>

#include "rlkv_host.cuh"

using namespace rlkv;

namespace rlkv {
thread_local char g_cuda_text[256] = "";
}

namespace {

struct Layout {
    int rows_full = 0, rows_comp = 0;
    std::vector<int> n_full, n_comp;
    std::vector<long long> full_row0, comp_row0;  // per layer, in pool rows
    long long pool_rows = 0;
    size_t off_layer_desc = 0;
    size_t off_pool = 0, off_tables = 0, off_tickets = 0, off_status = 0, off_partials = 0;
    size_t off_k = 0, off_v = 0, off_q = 0, off_out = 0, off_in2 = 0, off_trace = 0, total = 0;
    int max_grid = 0, max_items = 0;
    bool step_in_one_launch = false;  // the shape allows rlkv_step to serve all layers with one decode launch
};

constexpr int kDefaultItemTilesAlone = 8;    // a launch on its own: finer items for an even finish
constexpr int kMaxFanIn = 32;                // most pieces a full unit is cut into when the schedule has no bands

int check_shape(int layers, int kv_heads, int q_heads, int head_dim, int batch, int max_len,
                const uint8_t* mask, int sink, int window)
{
    if (!mask || layers < 1 || kv_heads < 1 || kv_heads > kMaxKvHeads || q_heads < 1 || batch < 1 || max_len < 1)
        return RLKV_EINVAL;
    if (q_heads % kv_heads != 0 || q_heads / kv_heads > kMaxGroup) return RLKV_EINVAL;
    if (head_dim != 64 && head_dim != 128) return RLKV_EINVAL;
    if (sink < 0 || window < 1) return RLKV_EINVAL;
    if ((long long)sink + window > (1 << 24) || max_len > (1 << 28)) return RLKV_EINVAL;
    return RLKV_OK;
}

int make_layout(Layout& L, int layers, int kv_heads, int q_heads, int head_dim, int batch, int max_len,
                const uint8_t* mask, int sink, int window)
{
    L.rows_full = (int)align_up((size_t)max_len, kTile);
    L.rows_comp = (int)align_up((size_t)sink + window, kTile);
    L.n_full.assign(layers, 0);
    L.n_comp.assign(layers, 0);
    L.full_row0.assign(layers, 0);
    L.comp_row0.assign(layers, 0);
    long long row = 0;
    for (int l = 0; l < layers; ++l) {
        for (int h = 0; h < kv_heads; ++h) (mask[l * kv_heads + h] ? L.n_full[l] : L.n_comp[l])++;
        L.full_row0[l] = row;
        row += (long long)batch * L.n_full[l] * 2 * L.rows_full;
        L.comp_row0[l] = row;
        row += (long long)batch * L.n_comp[l] * 2 * L.rows_comp;
    }
    L.pool_rows = row;
    if (row >= (1ll << 31)) return RLKV_EINVAL;  // TMA row coordinates are 32-bit
    L.max_grid = 2 * kMaxGridSms;
    {
        // partial records: sized for the layer and length that can need the most of them
        long long most = 0;
        for (int l = 0; l < layers; ++l) {
            const long long t = (long long)batch * (L.n_full[l] * (long long)(L.rows_full / kTile) +
                                                    L.n_comp[l] * (long long)(L.rows_comp / kTile));
            if (t >= (1ll << 31)) return RLKV_EINVAL;
            const long long m = most_slots(batch * L.n_full[l], L.rows_full / kTile, batch * L.n_comp[l],
                                           L.rows_comp / kTile, L.max_grid);
            if (m > most) most = m;
            if (L.n_comp[l] == 0) {  // a layer rlkv_decode_mixed_attention accepts: a local unit beside every full unit
                const int local_tiles = (sink + kTile - 1) / kTile + (window + kTile - 1) / kTile;
                const long long mm = most_slots(batch * L.n_full[l], L.rows_full / kTile, batch * L.n_full[l], local_tiles,
                                                L.max_grid);
                if (mm > most) most = mm;
            }
        }
        // a whole step in one launch (step_schedule) uses both halves of the scratch as one: its prefix
        // gives every CTA and every full unit at most one record, the rest is cut into items of at least
        // kMinItemTiles tiles while the step is small and of kDefaultItemTiles tiles once it is large
        {
            long long U = 0, Uc = 0;
            for (int l = 0; l < layers; ++l) {
                U += (long long)batch * L.n_full[l];
                Uc += (long long)batch * L.n_comp[l];
            }
            const long long T = U * (L.rows_full / kTile) + Uc * (L.rows_comp / kTile);
            const long long small = (long long)L.max_grid * kDefaultItemTiles / kMinItemTiles + 1;  // T < grid * 32
            const long long large = T / kDefaultItemTiles + 1;
            const long long fused = 2ll * L.max_grid + 2 * U + Uc + (small > large ? small : large) + 8;
            L.step_in_one_launch = layers <= kMaxStepLayers && layers * kv_heads <= kMaxStepHeads && T < (1ll << 31) &&
                                   fused < (1ll << 31);
            if (L.step_in_one_launch && (fused + 1) / 2 > most) most = (fused + 1) / 2;
        }
        if (most >= (1ll << 31)) return RLKV_EINVAL;
        L.max_items = (int)most;
    }
    size_t off = 0;
    L.off_pool = off;
    off = align_up(off + (size_t)row * head_dim * 2, 1024);
    L.off_tables = off;
    off = align_up(off + (size_t)2 * layers * kv_heads * sizeof(int), 16);
    L.off_layer_desc = off;
    off = align_up(off + (size_t)layers * sizeof(LayerDesc), 1024);
    L.off_tickets = off;
    off = align_up(off + (size_t)layers * 2 * batch * kv_heads * sizeof(int), 1024);
    L.off_status = off;
    off = align_up(off + 64, 1024);
    L.off_partials = off;
    off = align_up(off + (size_t)2 * L.max_items * partial_floats(head_dim, q_heads / kv_heads) * sizeof(float), 1024);
    const size_t kv_step = (size_t)layers * batch * kv_heads * head_dim * 2;
    const size_t q_step = (size_t)layers * batch * q_heads * head_dim * 2;
    L.off_k = off;
    off = align_up(off + kv_step, 1024);
    L.off_v = off;
    off = align_up(off + kv_step, 1024);
    L.off_q = off;
    off = align_up(off + q_step, 1024);
    L.off_out = off;
    off = align_up(off + q_step * 2, 1024);
    L.off_in2 = off;  // second copy of the k, v, q staging (same internal layout as the first)
    off = align_up(off + (L.off_out - L.off_k), 1024);
    L.off_trace = off;
    off = align_up(off + (size_t)L.max_grid * kTraceWords * sizeof(unsigned long long), 1024);
    L.total = off;
    return RLKV_OK;
}

}  // namespace

struct rlkv_cache {
    int layers, kv_heads, q_heads, head_dim, batch, max_len, sink, window;
    int device, sm_count;
    int ctas_per_sm, stages, groups, item_tiles;  // decode launch shape (rlkv_set_decode_config)
    int item_tiles_alone;                         // item_tiles of launches outside rlkv_step
    int trace_on;
    int out_bf16;            // results are stored as bf16 instead of fp32 (rlkv_set_output_bf16)
    int step_mode;           // rlkv_step: 0 chooses, 1 one decode launch per layer, 2 one for the whole step
    StepArgs step_args;      // the layer tables of a whole-step launch
    unsigned int claims[2];  // value of each work-claim counter after the launches issued so far
    cudaStream_t in_stream, out_stream;  // rlkv_step_host: copies that run beside the kernels
    cudaEvent_t ev_step[2], ev_done;     // kernels of a call done with staging copy p / results copied out
    cudaEvent_t ev_in[4], ev_out[4];     // per chunk of layers: its inputs have arrived / its results are ready
    unsigned long long host_steps;       // rlkv_step_host calls so far
    Layout lay;
    std::vector<uint8_t> is_full;
    std::vector<int> slot_of_head, head_of_slot;  // [layers*kv_heads]
    std::vector<int> len;                         // [layers]
    uint8_t* dev_base;
    bool owns_buffer;
    CUtensorMap tmap;
    uint64_t launches;
    // A cache created by rlkv_cache_create_fp8 keeps its K/V rows as 8-bit codes in a paged cache of
    // `batch` request slots whose pages are handed out in order (fp8_* below): every call is passed on to
    // it, and none of the device members above is used.
    rlkv_paged* fp8;
    std::vector<int> fp8_slots;   // the request slot of every batch row
    uint8_t* fp8_staging;         // k, v, q, out of one step, for rlkv_step_host
};

namespace {

void destroy_copy_objects(rlkv_cache* c)
{
    if (c->in_stream) cudaStreamDestroy(c->in_stream);
    if (c->out_stream) cudaStreamDestroy(c->out_stream);
    if (c->ev_step[0]) cudaEventDestroy(c->ev_step[0]);
    if (c->ev_step[1]) cudaEventDestroy(c->ev_step[1]);
    if (c->ev_done) cudaEventDestroy(c->ev_done);
    for (int i = 0; i < 4; ++i) {
        if (c->ev_in[i]) cudaEventDestroy(c->ev_in[i]);
        if (c->ev_out[i]) cudaEventDestroy(c->ev_out[i]);
    }
    c->in_stream = c->out_stream = nullptr;
}

template <typename T>
T* dev_at(const rlkv_cache* c, size_t off) { return reinterpret_cast<T*>(c->dev_base + off); }

int zero_state(rlkv_cache* c, cudaStream_t s)
{
    // pools, tickets and status; tables and the rest need no clearing
    RLKV_CUDA(cudaMemsetAsync(c->dev_base + c->lay.off_pool, 0, (size_t)c->lay.pool_rows * c->head_dim * 2, s));
    RLKV_CUDA(cudaMemsetAsync(c->dev_base + c->lay.off_tickets, 0,
                              c->lay.off_partials - c->lay.off_tickets, s));
    return RLKV_OK;
}

int make_tensor_map(rlkv_cache* c)
{
    return encode_pool_tensor_map(&c->tmap, c->dev_base + c->lay.off_pool, c->lay.pool_rows, c->head_dim);
}

bool valid_layer(const rlkv_cache* c, int layer) { return c && layer >= 0 && layer < c->layers; }

int do_append(rlkv_cache* c, int layer, const void* k, const void* v, int n_tokens, cudaStream_t s, bool overlap = false)
{
    AppendArgs a;
    a.overlap = overlap ? 1 : 0;
    a.pool = dev_at<__nv_bfloat16>(c, c->lay.off_pool);
    a.full_row0 = c->lay.full_row0[layer];
    a.comp_row0 = c->lay.comp_row0[layer];
    a.slot_of_head = dev_at<int>(c, c->lay.off_tables) + (size_t)layer * c->kv_heads;
    a.k = static_cast<const __nv_bfloat16*>(k);
    a.v = static_cast<const __nv_bfloat16*>(v);
    a.n_full = c->lay.n_full[layer];
    a.n_comp = c->lay.n_comp[layer];
    a.rows_full = c->lay.rows_full;
    a.rows_comp = c->lay.rows_comp;
    a.batch = c->batch;
    a.kv_heads = c->kv_heads;
    a.head_dim = c->head_dim;
    a.t0 = c->len[layer];
    a.n_tokens = n_tokens;
    a.sink = c->sink;
    a.window = c->window;
    RLKV_CUDA(launch_append(a, s));
    c->launches++;
    c->len[layer] += n_tokens;
    return RLKV_OK;
}

// Everything of a decode launch except where its split-KV work area lives.  Returns the grid size
// in *grid_out.
// `alpha` != null: a mixed-attention launch (every head of the layer is full, and the layer holds more
// than sink + window tokens): the first class of units covers the tokens between the sink and the
// window, the second class are the local units, one per (batch row, head), over the head's sink and
// window rows.  No row is read twice: the full branch of Eq. 1 merges both units' records.
int build_decode_args(rlkv_cache* c, int layer, const void* q, void* out, DecodeArgs& a, int* grid_out,
                      bool in_step = false, const float* alpha = nullptr)
{
    const int n = c->len[layer];
    const int cap = c->sink + c->window;
    a.pool = dev_at<__nv_bfloat16>(c, c->lay.off_pool);
    a.full_row0 = c->lay.full_row0[layer];
    a.comp_row0 = c->lay.comp_row0[layer];
    for (int h = 0; h < c->kv_heads; ++h) a.head_of_slot[h] = (unsigned char)c->head_of_slot[(size_t)layer * c->kv_heads + h];
    a.q = static_cast<const __nv_bfloat16*>(q);
    a.out = static_cast<float*>(out);
    a.status = dev_at<int>(c, c->lay.off_status);
    a.trace = dev_at<unsigned long long>(c, c->lay.off_trace);
    a.n_full = c->lay.n_full[layer];
    a.n_comp = c->lay.n_comp[layer];
    a.rows_full = c->lay.rows_full;
    a.rows_comp = c->lay.rows_comp;
    a.len_full = n;
    a.len_comp = n < cap ? n : cap;
    a.batch = c->batch;
    a.group = c->q_heads / c->kv_heads;
    a.q_heads = c->q_heads;
    a.alpha = alpha;
    a.new_k = a.new_v = nullptr;
    a.new_sink = c->sink;
    a.new_window = c->window;
    a.local_sink = n < c->sink ? n : c->sink;
    a.local_sink_tiles = (a.local_sink + kTile - 1) / kTile;
    a.local_win0 = n - c->window > c->sink ? n - c->window : c->sink;  // first token of the window
    a.local_win_len = n > a.local_win0 ? n - a.local_win0 : 0;
    if (alpha) a.len_full = n - c->window - c->sink;  // > 0: the caller sends shorter layers to the plain kernel
    const int tiles_full = (a.len_full + kTile - 1) / kTile;
    const int tiles_comp = alpha ? a.local_sink_tiles + (a.local_win_len + kTile - 1) / kTile : (a.len_comp + kTile - 1) / kTile;
    const int second_class = alpha ? a.n_full : a.n_comp;  // units per batch row beside the full ones
    const long long all_tiles = (long long)c->batch * ((long long)a.n_full * tiles_full + (long long)second_class * tiles_comp);
    if (all_tiles >= (1ll << 31)) return RLKV_EINVAL;
    a.scale_log2 = 1.4426950408889634f / sqrtf((float)c->head_dim);
    a.trace_on = c->trace_on;
    a.out_bf16 = c->out_bf16;
    // persistent grid; the work items of the flat tile space are cut for that many CTAs and no
    // more CTAs are launched than there are items
    int grid = c->sm_count * c->ctas_per_sm;
    if (grid > c->lay.max_grid) grid = c->lay.max_grid;
    // smallest work item: the configured size, less where the launch is too small to give every CTA
    // one item of that size
    int item_tiles = (int)(all_tiles / (1ll * grid));
    const int most = in_step ? c->item_tiles : c->item_tiles_alone;
    if (item_tiles > most) item_tiles = most;
    if (item_tiles < kMinItemTiles) item_tiles = kMinItemTiles;
    a.sched = make_schedule(c->batch * a.n_full, tiles_full, c->batch * second_class, tiles_comp, grid, item_tiles);
    // A launch too small for the schedule to form bands cuts every full unit into tiles_full / item_tiles
    // pieces, all merged by one CTA at the end: with a few long rows that fan-in, not the bytes, sets
    // the time.  Larger items (fewer CTAs, each streaming longer) bound it.
    // Inside a step only where the launch would not fill the GPU anyway: a full grid overlaps with its
    // neighbours, which hides the merge better than larger items avoid it.
    if (a.sched.R == 0 && a.n_full > 0 && tiles_full > kMaxFanIn * item_tiles && (!in_step || a.sched.n_items < grid)) {
        item_tiles = (tiles_full + kMaxFanIn - 1) / kMaxFanIn;
        a.sched = make_schedule(c->batch * a.n_full, tiles_full, c->batch * second_class, tiles_comp, grid, item_tiles);
    }
    if (grid > a.sched.n_items) grid = a.sched.n_items;
    *grid_out = grid;
    return RLKV_OK;
}

// `half`: which half of the scratch memory (partials, claim counter) the launch uses; `overlap` and
// `dep_wait` as in launch_decode.
int do_decode(rlkv_cache* c, int layer, const void* q, void* out, cudaStream_t s, int half = 0, bool overlap = false,
              int dep_wait = 0, int* grid_out = nullptr, const float* alpha = nullptr, bool in_step = false,
              const void* new_k = nullptr, const void* new_v = nullptr)
{
    DecodeArgs a;
    int grid = 0;
    int rc = build_decode_args(c, layer, q, out, a, &grid, in_step, alpha);
    if (rc) return rc;
    a.new_k = static_cast<const __nv_bfloat16*>(new_k);  // the launch appends the token itself (len already counts it)
    a.new_v = static_cast<const __nv_bfloat16*>(new_v);
    if (a.sched.n_slots > c->lay.max_items) return RLKV_ESCRATCH;  // cannot happen: the scratch is sized for it
    a.partials = dev_at<float>(c, c->lay.off_partials) +
                 (size_t)half * c->lay.max_items * partial_floats(c->head_dim, a.group);
    a.tickets = dev_at<int>(c, c->lay.off_tickets) + (size_t)layer * 2 * c->batch * c->kv_heads;
    a.claim_counter = dev_at<unsigned int>(c, c->lay.off_status) + 4 + half;
    a.claim_base = c->claims[half];
    a.dep_wait = dep_wait;
    RLKV_CUDA(launch_decode(a, &c->tmap, c->head_dim, grid, c->stages, c->groups, s, overlap, alpha ? kModeMixed : kModePlain));
    c->claims[half] += (unsigned int)a.sched.n_items;  // every CTA claims until it is told there is no more
    if (grid_out) *grid_out = grid;
    c->launches++;
    return RLKV_OK;
}

// One decode launch for layers [l0, l1) of a step (all of them hold the same number of tokens).  q, out:
// the step's [layers][batch][q_heads][head_dim] arrays.  `after_append`: the launch directly follows the
// step's append launch and may start beside it; otherwise it is an ordinary launch.  Launches of this
// kind never overlap one another, so each uses the whole split-KV scratch.
int do_decode_step(rlkv_cache* c, int l0, int l1, const void* q, void* out, cudaStream_t s, bool after_append)
{
    const int n = c->len[l0];
    const int cap = c->sink + c->window;
    DecodeArgs a;
    memset(&a, 0, sizeof a);
    a.pool = dev_at<__nv_bfloat16>(c, c->lay.off_pool);
    const size_t q_layer = (size_t)c->batch * c->q_heads * c->head_dim;
    a.q = static_cast<const __nv_bfloat16*>(q) + l0 * q_layer;
    a.out = reinterpret_cast<float*>(static_cast<uint8_t*>(out) + l0 * q_layer * (c->out_bf16 ? 2 : 4));
    a.status = dev_at<int>(c, c->lay.off_status);
    a.trace = dev_at<unsigned long long>(c, c->lay.off_trace);
    a.rows_full = c->lay.rows_full;
    a.rows_comp = c->lay.rows_comp;
    a.len_full = n;
    a.len_comp = n < cap ? n : cap;
    a.batch = c->batch * (l1 - l0);
    a.group = c->q_heads / c->kv_heads;
    a.q_heads = c->q_heads;
    a.scale_log2 = 1.4426950408889634f / sqrtf((float)c->head_dim);
    a.trace_on = c->trace_on;
    a.out_bf16 = c->out_bf16;
    StepArgs part;                      // the tables of layers l0 .. l1-1, units counted from the first of them
    const StepArgs* stp = &c->step_args;
    if (l0 != 0 || l1 != c->layers) {
        const StepArgs& all = c->step_args;
        memset(&part, 0, sizeof part);
        part.head_of_slot = all.head_of_slot + (size_t)l0 * c->kv_heads;
        part.n_layers = l1 - l0;
        part.kv_heads = all.kv_heads;
        part.batch = all.batch;
        for (int l = l0; l <= l1; ++l) {
            part.full_base[l - l0] = all.full_base[l] - all.full_base[l0];
            part.comp_base[l - l0] = all.comp_base[l] - all.comp_base[l0];
            if (l < l1) {
                part.full_row0[l - l0] = all.full_row0[l];
                part.comp_row0[l - l0] = all.comp_row0[l];
            }
        }
        stp = &part;
    }
    const StepArgs& st = *stp;
    const int U = st.full_base[l1 - l0], Uc = st.comp_base[l1 - l0];
    const int tiles_full = (a.len_full + kTile - 1) / kTile, tiles_comp = (a.len_comp + kTile - 1) / kTile;
    if ((long long)U * tiles_full + (long long)Uc * tiles_comp >= (1ll << 31)) return RLKV_EINVAL;
    int grid = c->sm_count * c->ctas_per_sm;
    if (grid > c->lay.max_grid) grid = c->lay.max_grid;
    // the scratch is sized for items of kDefaultItemTiles tiles once the step is large: a smaller setting
    // (rlkv_set_decode_config) is raised until the partial records fit
    int item_most = c->item_tiles;
    a.sched = step_schedule(U, tiles_full, Uc, tiles_comp, grid, item_most);
    while (a.sched.n_slots > 2 * c->lay.max_items && item_most < kDefaultItemTiles) {
        item_most = item_most * 2 < kDefaultItemTiles ? item_most * 2 : kDefaultItemTiles;
        a.sched = step_schedule(U, tiles_full, Uc, tiles_comp, grid, item_most);
    }
    if (grid > a.sched.n_items) grid = a.sched.n_items;
    if (a.sched.n_slots > 2 * c->lay.max_items) return RLKV_ESCRATCH;  // cannot happen: the scratch is sized for it
    a.partials = dev_at<float>(c, c->lay.off_partials);                // both halves as one
    a.tickets = dev_at<int>(c, c->lay.off_tickets) + (size_t)l0 * 2 * c->batch * c->kv_heads;  // one per unit of the launch
    a.claim_counter = dev_at<unsigned int>(c, c->lay.off_status) + 4;
    a.claim_base = c->claims[0];
    a.dep_wait = after_append ? 1 : 0;
    RLKV_CUDA(launch_decode(a, &c->tmap, c->head_dim, grid, c->stages, c->groups, s, after_append, kModeStep, nullptr, nullptr,
                            &st));
    c->claims[0] += (unsigned int)a.sched.n_items;
    c->launches++;
    return RLKV_OK;
}

// Whether rlkv_step serves all layers with one decode launch: the shape must allow it and every layer
// must hold the same number of tokens; left to the library (step_mode 0) it is chosen always -- one
// flat tile space over all layers has no per-layer start-up, tail or merge phase to hide.
bool step_uses_one_launch(const rlkv_cache* c)
{
    if (c->step_mode == 1 || !c->lay.step_in_one_launch) return false;
    for (int l = 1; l < c->layers; ++l)
        if (c->len[l] != c->len[0]) return false;
    return true;
}

// ---- split-KV scratch that nobody allocates -------------------------------------------------------
// rlkv_decode_attention_static_scratch keeps the decode kernel's split bookkeeping (work-claim
// counters, tickets) and partial results here instead of in the cache's own buffer.  The array is
// part of the library image: every GPU that loads librlkv holds these bytes until the process exits.
constexpr size_t kStaticScratchBytes = 4u << 20;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
// device address of the array, per device; two host threads that make their first call on a device at
// the same time both ask the runtime and store the same answer
std::atomic<unsigned char*> g_static_scratch_dev[kMaxDevices];

// Device address of g_static_scratch on `device`, which must be current.  In host code the array's
// name is only a handle for the runtime, never a pointer a kernel may use: the address has to be
// asked for, once per device.
int static_scratch_address(int device, unsigned char** out)
{
    if (device < 0 || device >= kMaxDevices) return RLKV_EINVAL;
    unsigned char* known = g_static_scratch_dev[device].load(std::memory_order_acquire);
    if (!known) {
        void* p = nullptr;
        RLKV_CUDA(cudaGetSymbolAddress(&p, g_static_scratch));
        if (!p) return cuda_fail(cudaErrorInvalidSymbol, "cudaGetSymbolAddress(g_static_scratch)");
        known = static_cast<unsigned char*>(p);
        g_static_scratch_dev[device].store(known, std::memory_order_release);
    }
    *out = known;
    return RLKV_OK;
}

// The launch of do_decode with counters, tickets and partials placed in the static array.
int do_decode_static_scratch(rlkv_cache* c, int layer, const void* q, void* out, cudaStream_t s)
{
    DecodeArgs a;
    int grid = 0;
    int rc = build_decode_args(c, layer, q, out, a, &grid);
    if (rc) return rc;
    // carve the static array: the two counters and one ticket per (batch row, KV head), then the
    // partial records of this launch
    const size_t head_bytes = align_up((2 + (size_t)c->batch * c->kv_heads) * sizeof(int), 256);  // claim counter, tickets
    const size_t partial_bytes = (size_t)a.sched.n_slots * partial_floats(c->head_dim, a.group) * sizeof(float);
    if (head_bytes + partial_bytes > kStaticScratchBytes) return RLKV_ESCRATCH;
    unsigned char* base = nullptr;
    rc = static_scratch_address(c->device, &base);
    if (rc) return rc;
    a.claim_counter = reinterpret_cast<unsigned int*>(base);
    a.claim_base = 0;
    a.dep_wait = 0;
    a.tickets = reinterpret_cast<int*>(base) + 2;
    a.partials = reinterpret_cast<float*>(base + head_bytes);
    // the array still holds whatever the previous call (of any cache) left: counters and tickets
    // must start at zero
    RLKV_CUDA(cudaMemsetAsync(base, 0, head_bytes, s));
    RLKV_CUDA(launch_decode(a, &c->tmap, c->head_dim, grid, c->stages, c->groups, s, false));
    c->launches++;
    return RLKV_OK;
}

// The launches of one decode step on device buffers (k, v, q, out as in rlkv_step).
// step_append: one launch appends the new token to every layer.  step_decode: the decode launches of
// layers [l0, l1).  All inputs of the step are complete before its first launch starts, so the decode
// launches may overlap one another: consecutive layers alternate between the two halves of the
// scratch memory, the first layer's launch waits on the device for the append launch before it reads
// rows that launch writes, and every later launch lets its successor start only after its own
// predecessor has completed (step_launch_mode in rlkv_host.cuh), so two launches that share a half are
// never in flight together.  After anything but a kernel of this step in the stream (`fresh`) the
// first launch is an ordinary one, which waits for everything before it.
int step_append(rlkv_cache* c, const void* k, const void* v, cudaStream_t s)
{
    AppendAllArgs aa;
    aa.pool = dev_at<__nv_bfloat16>(c, c->lay.off_pool);
    aa.layers = dev_at<LayerDesc>(c, c->lay.off_layer_desc);
    aa.slot_of_head = dev_at<int>(c, c->lay.off_tables);
    aa.k = static_cast<const __nv_bfloat16*>(k);
    aa.v = static_cast<const __nv_bfloat16*>(v);
    aa.n_layers = c->layers;
    aa.rows_full = c->lay.rows_full;
    aa.rows_comp = c->lay.rows_comp;
    aa.batch = c->batch;
    aa.kv_heads = c->kv_heads;
    aa.head_dim = c->head_dim;
    aa.sink = c->sink;
    aa.window = c->window;
    for (int l = 0; l < c->layers; ++l) aa.t0[l] = c->len[l];
    RLKV_CUDA(launch_append_all(aa, s));
    c->launches++;
    for (int l = 0; l < c->layers; ++l) c->len[l] += 1;
    return RLKV_OK;
}

int step_decode(rlkv_cache* c, int l0, int l1, const void* q, void* out, cudaStream_t s, bool fresh)
{
    const size_t q_layer = (size_t)c->batch * c->q_heads * c->head_dim;
    for (int l = l0; l < l1; ++l) {
        const StepLaunchMode m = step_launch_mode(l == l0, !fresh && l == 0);
        int rc = do_decode(c, l, static_cast<const __nv_bfloat16*>(q) + l * q_layer,
                           static_cast<uint8_t*>(out) + l * q_layer * (c->out_bf16 ? 2 : 4), s, l & 1, m.overlap, m.dep_wait,
                           nullptr, nullptr, true);
        if (rc) return rc;
    }
    return RLKV_OK;
}

// ---- the lock-step cache kept in 8 bits: a thin layer over the paged cache ------------------------
int fp8_prefill(rlkv_cache* c, int layer, const void* k, const void* v, int n_tokens, void* stream)
{
    if ((long long)c->len[layer] + n_tokens > c->max_len) return RLKV_EFULL;
    const long long row = (long long)c->kv_heads * c->head_dim;
    if (n_tokens == 1) {
        const int rc = rlkv_paged_append(c->fp8, layer, c->fp8_slots.data(), c->batch, k, v, stream);
        if (rc == RLKV_OK) c->len[layer] += 1;
        return rc;
    }
    for (int b = 0; b < c->batch; ++b) {  // batch row b's tokens lie batch * kv_heads * head_dim elements apart
        const int rc = paged_prefill_strided(c->fp8, layer, c->fp8_slots[b], static_cast<const __nv_bfloat16*>(k) + b * row,
                                             static_cast<const __nv_bfloat16*>(v) + b * row, n_tokens, c->batch * row, stream);
        if (rc) return rc;
    }
    c->len[layer] += n_tokens;
    return RLKV_OK;
}

int fp8_step(rlkv_cache* c, const void* k, const void* v, const void* q, void* out, void* stream)
{
    const int rc = rlkv_paged_step(c->fp8, c->fp8_slots.data(), c->batch, k, v, q, out, stream);
    if (rc == RLKV_OK)
        for (int l = 0; l < c->layers; ++l) c->len[l] += 1;
    return rc;
}

int fp8_export(rlkv_cache* c, int layer, int b, int h, void* k_host, void* v_host, int* rows_out, int32_t* token_of_slot)
{
    // the paged export gives a full head's rows in token order, which is this cache's physical order;
    // rows that hold no token are reported as zeros
    const bool full = c->is_full[(size_t)layer * c->kv_heads + h] != 0;
    const int rows = full ? c->max_len : c->sink + c->window;
    memset(k_host, 0, (size_t)rows * c->head_dim * 2);
    memset(v_host, 0, (size_t)rows * c->head_dim * 2);
    for (int s = 0; s < rows; ++s) token_of_slot[s] = -1;
    int got = 0;
    const int rc = rlkv_paged_debug_export_head(c->fp8, layer, c->fp8_slots[b], h, k_host, v_host, &got, token_of_slot);
    if (rc) return rc;
    for (int s = 0; s < rows; ++s)  // a ring slot no token has reached since the reset may hold older codes
        if (token_of_slot[s] < 0) {
            memset(static_cast<uint8_t*>(k_host) + (size_t)s * c->head_dim * 2, 0, (size_t)c->head_dim * 2);
            memset(static_cast<uint8_t*>(v_host) + (size_t)s * c->head_dim * 2, 0, (size_t)c->head_dim * 2);
        }
    *rows_out = rows;
    return RLKV_OK;
}

}  // namespace

extern "C" {

const char* rlkv_strerror(int code)
{
    switch (code) {
        case RLKV_OK: return "ok";
        case RLKV_EINVAL: return "invalid argument";
        case RLKV_EFULL: return "cache is at max_len";
        case RLKV_EEMPTY: return "layer holds no token";
        case RLKV_ENOMEM: return "out of memory or buffer too small";
        case RLKV_ECUDA: return g_cuda_text[0] ? g_cuda_text : "CUDA error";
        case RLKV_EKERNEL: return "a kernel gave up on a bounded wait";
        case RLKV_ESCRATCH: return "the launch needs more scratch than the library's static array holds";
        default: return "unknown error";
    }
}

int rlkv_cache_size(int layers, int kv_heads, int q_heads, int head_dim, int batch, int max_len,
                    const uint8_t* head_is_full, int sink, int window, size_t* bytes_out)
{
    if (!bytes_out) return RLKV_EINVAL;
    int rc = check_shape(layers, kv_heads, q_heads, head_dim, batch, max_len, head_is_full, sink, window);
    if (rc) return rc;
    Layout L;
    rc = make_layout(L, layers, kv_heads, q_heads, head_dim, batch, max_len, head_is_full, sink, window);
    if (rc) return rc;
    *bytes_out = L.total;
    return RLKV_OK;
}

int rlkv_cache_create(rlkv_cache** out, int layers, int kv_heads, int q_heads, int head_dim, int batch,
                      int max_len, const uint8_t* head_is_full, int sink, int window, void* device_buf,
                      size_t device_buf_bytes)
{
    if (!out) return RLKV_EINVAL;
    *out = nullptr;
    int rc = check_shape(layers, kv_heads, q_heads, head_dim, batch, max_len, head_is_full, sink, window);
    if (rc) return rc;
    rlkv_cache* c = new (std::nothrow) rlkv_cache();
    if (!c) return RLKV_ENOMEM;
    c->layers = layers; c->kv_heads = kv_heads; c->q_heads = q_heads; c->head_dim = head_dim;
    c->batch = batch; c->max_len = max_len; c->sink = sink; c->window = window;
    c->dev_base = nullptr; c->owns_buffer = false; c->launches = 0;
    c->ctas_per_sm = 1;
    c->groups = 2;
    c->item_tiles = kDefaultItemTiles;
    c->item_tiles_alone = kDefaultItemTilesAlone;
    c->trace_on = 0;
    c->out_bf16 = 0;
    c->step_mode = 0;
    c->fp8 = nullptr;
    c->fp8_staging = nullptr;
    c->claims[0] = c->claims[1] = 0;
    c->in_stream = c->out_stream = nullptr;
    c->ev_step[0] = c->ev_step[1] = c->ev_done = nullptr;
    c->host_steps = 0;
    for (int i = 0; i < 4; ++i) c->ev_in[i] = c->ev_out[i] = nullptr;
    c->stages = max_stages(head_dim, q_heads / kv_heads, c->groups, c->ctas_per_sm);
    rc = make_layout(c->lay, layers, kv_heads, q_heads, head_dim, batch, max_len, head_is_full, sink, window);
    if (rc) { delete c; return rc; }
    c->is_full.assign(head_is_full, head_is_full + (size_t)layers * kv_heads);
    c->len.assign(layers, 0);
    c->slot_of_head.assign((size_t)layers * kv_heads, 0);
    c->head_of_slot.assign((size_t)layers * kv_heads, 0);
    for (int l = 0; l < layers; ++l) {
        int nf = 0, nc = 0;
        for (int h = 0; h < kv_heads; ++h) {
            if (c->is_full[l * kv_heads + h]) {
                c->slot_of_head[l * kv_heads + h] = nf;
                c->head_of_slot[l * kv_heads + nf] = h;
                ++nf;
            } else {
                c->slot_of_head[l * kv_heads + h] = -(nc + 1);
                ++nc;
            }
        }
        nc = 0;
        for (int h = 0; h < kv_heads; ++h)
            if (!c->is_full[l * kv_heads + h]) c->head_of_slot[l * kv_heads + nf + nc++] = h;
    }
    auto fail = [&](int code) {
        destroy_copy_objects(c);
        if (c->owns_buffer && c->dev_base) cudaFree(c->dev_base);
        delete c;
        return code;
    };
    cudaError_t e = cudaGetDevice(&c->device);
    if (e != cudaSuccess) return fail(cuda_fail(e, "cudaGetDevice"));
    e = cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, c->device);
    if (e != cudaSuccess) return fail(cuda_fail(e, "cudaDeviceGetAttribute"));
    if (c->sm_count > kMaxGridSms) c->sm_count = kMaxGridSms;
    if (device_buf) {
        if ((reinterpret_cast<uintptr_t>(device_buf) & 1023u) != 0) return fail(RLKV_EINVAL);
        if (device_buf_bytes < c->lay.total) return fail(RLKV_ENOMEM);
        c->dev_base = static_cast<uint8_t*>(device_buf);
    } else {
        void* p = nullptr;
        e = cudaMalloc(&p, c->lay.total);
        if (e != cudaSuccess) {
            cudaGetLastError();
            return fail(RLKV_ENOMEM);
        }
        c->dev_base = static_cast<uint8_t*>(p);
        c->owns_buffer = true;
    }
    rc = zero_state(c, nullptr);
    if (rc) return fail(rc);
    const size_t tbytes = (size_t)layers * kv_heads * sizeof(int);
    e = cudaMemcpy(c->dev_base + c->lay.off_tables, c->slot_of_head.data(), tbytes, cudaMemcpyHostToDevice);
    if (e == cudaSuccess)
        e = cudaMemcpy(c->dev_base + c->lay.off_tables + tbytes, c->head_of_slot.data(), tbytes,
                       cudaMemcpyHostToDevice);
    if (e == cudaSuccess) {
        std::vector<LayerDesc> desc(layers);
        for (int l = 0; l < layers; ++l)
            desc[l] = LayerDesc{c->lay.full_row0[l], c->lay.comp_row0[l], c->lay.n_full[l], c->lay.n_comp[l]};
        e = cudaMemcpy(c->dev_base + c->lay.off_layer_desc, desc.data(), desc.size() * sizeof(LayerDesc),
                       cudaMemcpyHostToDevice);
    }
    if (e != cudaSuccess) return fail(cuda_fail(e, "cudaMemcpy(tables)"));
    {
        StepArgs& st = c->step_args;
        memset(&st, 0, sizeof st);
        st.head_of_slot = reinterpret_cast<const int*>(c->dev_base + c->lay.off_tables + tbytes);
        st.n_layers = layers;
        st.kv_heads = kv_heads;
        st.batch = batch;
        if (c->lay.step_in_one_launch)
            for (int l = 0; l < layers; ++l) {
                st.full_base[l + 1] = st.full_base[l] + batch * c->lay.n_full[l];
                st.comp_base[l + 1] = st.comp_base[l] + batch * c->lay.n_comp[l];
                st.full_row0[l] = (int)c->lay.full_row0[l];
                st.comp_row0[l] = (int)c->lay.comp_row0[l];
            }
    }
    rc = make_tensor_map(c);
    if (rc) return fail(rc);
    e = prepare_decode_kernels(head_dim);
    if (e != cudaSuccess) return fail(cuda_fail(e, "cudaFuncSetAttribute"));
    e = cudaStreamCreateWithFlags(&c->in_stream, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&c->out_stream, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->ev_step[0], cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->ev_step[1], cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->ev_done, cudaEventDisableTiming);
    for (int i = 0; i < 4 && e == cudaSuccess; ++i) {
        e = cudaEventCreateWithFlags(&c->ev_in[i], cudaEventDisableTiming);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->ev_out[i], cudaEventDisableTiming);
    }
    if (e != cudaSuccess) return fail(cuda_fail(e, "cudaStreamCreate/cudaEventCreate"));
    e = cudaDeviceSynchronize();
    if (e != cudaSuccess) return fail(cuda_fail(e, "cudaDeviceSynchronize"));
    *out = c;
    return RLKV_OK;
}

namespace {
struct Fp8Sizes {
    size_t paged, kv, q, out, total;
};
int fp8_sizes(Fp8Sizes& z, int layers, int kv_heads, int q_heads, int head_dim, int batch, int max_len,
              const uint8_t* head_is_full, int sink, int window)
{
    int rc = check_shape(layers, kv_heads, q_heads, head_dim, batch, max_len, head_is_full, sink, window);
    if (rc) return rc;
    const int pages = batch * ((max_len + kTile - 1) / kTile);  // every row can reach max_len: no call ever finds the free list empty
    rc = rlkv_paged_size_fp8(layers, kv_heads, q_heads, head_dim, batch, pages, max_len, head_is_full, sink, window, &z.paged);
    if (rc) return rc;
    z.paged = align_up(z.paged, 1024);
    z.kv = align_up((size_t)layers * batch * kv_heads * head_dim * 2, 256);
    z.q = align_up((size_t)layers * batch * q_heads * head_dim * 2, 256);
    z.out = 2 * z.q;
    z.total = z.paged + 2 * z.kv + z.q + z.out;
    return RLKV_OK;
}
}  // namespace

int rlkv_cache_size_fp8(int layers, int kv_heads, int q_heads, int head_dim, int batch, int max_len,
                        const uint8_t* head_is_full, int sink, int window, size_t* bytes_out)
{
    if (!bytes_out) return RLKV_EINVAL;
    Fp8Sizes z;
    const int rc = fp8_sizes(z, layers, kv_heads, q_heads, head_dim, batch, max_len, head_is_full, sink, window);
    if (rc) return rc;
    *bytes_out = z.total;
    return RLKV_OK;
}

int rlkv_cache_create_fp8(rlkv_cache** out, int layers, int kv_heads, int q_heads, int head_dim, int batch,
                          int max_len, const uint8_t* head_is_full, int sink, int window, const float* k_scale,
                          const float* v_scale, void* device_buf, size_t device_buf_bytes)
{
    if (!out) return RLKV_EINVAL;
    *out = nullptr;
    if (!k_scale || !v_scale) return RLKV_EINVAL;
    Fp8Sizes z;
    int rc = fp8_sizes(z, layers, kv_heads, q_heads, head_dim, batch, max_len, head_is_full, sink, window);
    if (rc) return rc;
    rlkv_cache* c = new (std::nothrow) rlkv_cache();
    if (!c) return RLKV_ENOMEM;
    c->layers = layers; c->kv_heads = kv_heads; c->q_heads = q_heads; c->head_dim = head_dim;
    c->batch = batch; c->max_len = max_len; c->sink = sink; c->window = window;
    c->dev_base = nullptr; c->owns_buffer = false; c->launches = 0;
    c->trace_on = 0; c->out_bf16 = 0; c->step_mode = 0;
    c->fp8 = nullptr; c->fp8_staging = nullptr;
    c->in_stream = c->out_stream = nullptr;
    c->ev_step[0] = c->ev_step[1] = c->ev_done = nullptr;
    for (int i = 0; i < 4; ++i) c->ev_in[i] = c->ev_out[i] = nullptr;
    c->is_full.assign(head_is_full, head_is_full + (size_t)layers * kv_heads);
    c->len.assign(layers, 0);
    auto fail = [&](int code) {
        if (c->fp8) rlkv_paged_destroy(c->fp8);
        if (c->owns_buffer && c->dev_base) cudaFree(c->dev_base);
        delete c;
        return code;
    };
    cudaError_t e = cudaGetDevice(&c->device);
    if (e != cudaSuccess) return fail(cuda_fail(e, "cudaGetDevice"));
    if (device_buf) {
        if ((reinterpret_cast<uintptr_t>(device_buf) & 1023u) != 0) return fail(RLKV_EINVAL);
        if (device_buf_bytes < z.total) return fail(RLKV_ENOMEM);
        c->dev_base = static_cast<uint8_t*>(device_buf);
    } else {
        void* p = nullptr;
        e = cudaMalloc(&p, z.total);
        if (e != cudaSuccess) {
            cudaGetLastError();
            return fail(RLKV_ENOMEM);
        }
        c->dev_base = static_cast<uint8_t*>(p);
        c->owns_buffer = true;
    }
    c->fp8_staging = c->dev_base + z.paged;
    const int pages = batch * ((max_len + kTile - 1) / kTile);
    rc = rlkv_paged_create_fp8(&c->fp8, layers, kv_heads, q_heads, head_dim, batch, pages, max_len, head_is_full, sink,
                               window, k_scale, v_scale, c->dev_base, z.paged);
    if (rc) return fail(rc);
    c->fp8_slots.assign(batch, -1);
    for (int b = 0; b < batch; ++b) {
        rc = rlkv_paged_seq_open(c->fp8, &c->fp8_slots[b]);
        if (rc) return fail(rc);
    }
    *out = c;
    return RLKV_OK;
}

int rlkv_cache_destroy(rlkv_cache* c)
{
    if (!c) return RLKV_EINVAL;
    int rc = RLKV_OK;
    if (c->fp8) rc = rlkv_paged_destroy(c->fp8);  // synchronises the device; the buffer is this handle's
    {
        DeviceGuard g(c->device);
        destroy_copy_objects(c);
    }
    if (c->owns_buffer && c->dev_base) {
        DeviceGuard g(c->device);
        cudaError_t e = cudaFree(c->dev_base);
        if (e != cudaSuccess) rc = cuda_fail(e, "cudaFree");
    }
    delete c;
    return rc;
}

int rlkv_cache_reset(rlkv_cache* c, void* stream)
{
    if (!c) return RLKV_EINVAL;
    DeviceGuard g(c->device);
    if (!g.ok) return RLKV_ECUDA;
    if (c->fp8) {
        // Host bookkeeping only: every row's slot is closed (its pages go back to the free list) and
        // opened again.  Work enqueued later on the stream of the earlier calls runs after them.
        for (int b = 0; b < c->batch; ++b) {
            int rc = rlkv_paged_seq_close(c->fp8, c->fp8_slots[b]);
            if (rc) return rc;
        }
        for (int b = 0; b < c->batch; ++b) {
            int rc = rlkv_paged_seq_open(c->fp8, &c->fp8_slots[b]);
            if (rc) return rc;
        }
        std::fill(c->len.begin(), c->len.end(), 0);
        return RLKV_OK;
    }
    int rc = zero_state(c, static_cast<cudaStream_t>(stream));
    if (rc) return rc;
    std::fill(c->len.begin(), c->len.end(), 0);
    c->claims[0] = c->claims[1] = 0;  // zero_state has cleared the counters on the device
    return RLKV_OK;
}

int rlkv_set_decode_config(rlkv_cache* c, int ctas_per_sm, int stages, int consumer_groups, int item_tiles)
{
    if (c && c->fp8) return RLKV_EINVAL;  // the paged launches behind an 8-bit cache have one configuration
    if (!c || ctas_per_sm < 0 || ctas_per_sm > 2 || stages < 0 || stages == 1 || stages > 8 ||
        consumer_groups < 0 || consumer_groups > kMaxConsumerGroups ||
        (item_tiles != 0 && (item_tiles < kMinItemTiles || item_tiles > 1024)))
        return RLKV_EINVAL;
    const int cps = ctas_per_sm ? ctas_per_sm : c->ctas_per_sm;
    const int ng = consumer_groups ? consumer_groups : c->groups;
    const int most = max_stages(c->head_dim, c->q_heads / c->kv_heads, ng, cps);
    int st = stages ? stages : (c->stages < most ? c->stages : most);
    if (!stages) st -= st % ng;
    if (most < 2 || st < 2 || st > most || st % ng != 0) return RLKV_EINVAL;
    c->ctas_per_sm = cps;
    c->stages = st;
    c->groups = ng;
    if (item_tiles) c->item_tiles = c->item_tiles_alone = item_tiles;
    return RLKV_OK;
}

int rlkv_append(rlkv_cache* c, int layer, const void* k, const void* v, void* stream)
{
    return rlkv_prefill(c, layer, k, v, 1, stream);
}

int rlkv_prefill(rlkv_cache* c, int layer, const void* k, const void* v, int n_tokens, void* stream)
{
    if (!valid_layer(c, layer) || !k || !v || !aligned16(k) || !aligned16(v) || n_tokens < 1) return RLKV_EINVAL;
    if ((long long)c->len[layer] + n_tokens > c->max_len) return RLKV_EFULL;
    DeviceGuard g(c->device);
    if (!g.ok) return RLKV_ECUDA;
    if (c->fp8) return fp8_prefill(c, layer, k, v, n_tokens, stream);
    return do_append(c, layer, k, v, n_tokens, static_cast<cudaStream_t>(stream));
}

int rlkv_decode_attention(rlkv_cache* c, int layer, const void* q, void* out, void* stream)
{
    if (!valid_layer(c, layer) || !q || !out || !aligned16(q) || !aligned16(out)) return RLKV_EINVAL;
    if (c->len[layer] < 1) return RLKV_EEMPTY;
    DeviceGuard g(c->device);
    if (!g.ok) return RLKV_ECUDA;
    if (c->fp8) return rlkv_paged_decode_attention(c->fp8, layer, c->fp8_slots.data(), c->batch, q, out, stream);
    return do_decode(c, layer, q, out, static_cast<cudaStream_t>(stream));
}

int rlkv_append_overlapped(rlkv_cache* c, int layer, const void* k, const void* v, void* stream)
{
    if (!valid_layer(c, layer) || c->fp8 || !k || !v || !aligned16(k) || !aligned16(v)) return RLKV_EINVAL;
    if (c->len[layer] + 1 > c->max_len) return RLKV_EFULL;
    DeviceGuard g(c->device);
    if (!g.ok) return RLKV_ECUDA;
    return do_append(c, layer, k, v, 1, static_cast<cudaStream_t>(stream), true);
}

int rlkv_decode_attention_overlapped(rlkv_cache* c, int layer, const void* q, void* out, void* stream)
{
    if (!valid_layer(c, layer) || c->fp8 || !q || !out || !aligned16(q) || !aligned16(out)) return RLKV_EINVAL;
    if (c->len[layer] < 1) return RLKV_EEMPTY;
    DeviceGuard g(c->device);
    if (!g.ok) return RLKV_ECUDA;
    return do_decode(c, layer, q, out, static_cast<cudaStream_t>(stream), 0, true, 3);
}

int rlkv_layer_step_overlapped(rlkv_cache* c, int layer, const void* k, const void* v, const void* q, void* out, void* stream)
{
    if (!valid_layer(c, layer) || c->fp8 || !k || !v || !q || !out || !aligned16(k) || !aligned16(v) || !aligned16(q) ||
        !aligned16(out))
        return RLKV_EINVAL;
    if (c->len[layer] + 1 > c->max_len) return RLKV_EFULL;
    DeviceGuard g(c->device);
    if (!g.ok) return RLKV_ECUDA;
    c->len[layer] += 1;  // the launch writes the token's rows itself, each by the CTA that reads them
    const int rc = do_decode(c, layer, q, out, static_cast<cudaStream_t>(stream), 0, true, 3, nullptr, nullptr, false, k, v);
    if (rc) c->len[layer] -= 1;
    return rc;
}

int rlkv_decode_attention_static_scratch(rlkv_cache* c, int layer, const void* q, void* out, void* stream)
{
    if (!valid_layer(c, layer) || c->fp8 || !q || !out || !aligned16(q) || !aligned16(out)) return RLKV_EINVAL;
    if (c->len[layer] < 1) return RLKV_EEMPTY;
    DeviceGuard g(c->device);
    if (!g.ok) return RLKV_ECUDA;
    return do_decode_static_scratch(c, layer, q, out, static_cast<cudaStream_t>(stream));
}

size_t rlkv_static_scratch_bytes(void) { return kStaticScratchBytes; }

int rlkv_set_step_mode(rlkv_cache* c, int mode)
{
    if (!c || mode < 0 || mode > 2) return RLKV_EINVAL;
    if (c->fp8) return rlkv_paged_set_step_mode(c->fp8, mode);
    if (mode == 2 && !c->lay.step_in_one_launch) return RLKV_EINVAL;
    c->step_mode = mode;
    return RLKV_OK;
}

int rlkv_set_output_bf16(rlkv_cache* c, int on)
{
    if (!c) return RLKV_EINVAL;
    if (c->fp8) {
        const int rc = rlkv_paged_set_output_bf16(c->fp8, on);
        if (rc) return rc;
    }
    c->out_bf16 = on ? 1 : 0;
    return RLKV_OK;
}

int rlkv_decode_mixed_attention(rlkv_cache* c, int layer, const void* q, const float* alpha, void* out, void* stream)
{
    if (!valid_layer(c, layer) || c->fp8 || !q || !alpha || !out || !aligned16(q) || !aligned16(out)) return RLKV_EINVAL;
    if ((reinterpret_cast<uintptr_t>(alpha) & 3u) != 0) return RLKV_EINVAL;
    if (c->lay.n_comp[layer] != 0) return RLKV_EINVAL;  // the full branch needs every token of every head
    if (c->len[layer] < 1) return RLKV_EEMPTY;
    DeviceGuard g(c->device);
    if (!g.ok) return RLKV_ECUDA;
    // up to sink + window tokens every token is local: both branches of Eq. 1 are the plain attention
    if (c->len[layer] <= c->sink + c->window) return do_decode(c, layer, q, out, static_cast<cudaStream_t>(stream));
    return do_decode(c, layer, q, out, static_cast<cudaStream_t>(stream), 0, false, false, nullptr, alpha);
}

int rlkv_step(rlkv_cache* c, const void* k, const void* v, const void* q, void* out, void* stream)
{
    if (!c || !k || !v || !q || !out || !aligned16(k) || !aligned16(v) || !aligned16(q) || !aligned16(out))
        return RLKV_EINVAL;
    for (int l = 0; l < c->layers; ++l)
        if (c->len[l] >= c->max_len) return RLKV_EFULL;
    DeviceGuard g(c->device);
    if (!g.ok) return RLKV_ECUDA;
    if (c->fp8) return fp8_step(c, k, v, q, out, stream);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t kv_layer = (size_t)c->batch * c->kv_heads * c->head_dim;
    const size_t q_layer = (size_t)c->batch * c->q_heads * c->head_dim;
    if (c->layers <= kMaxStepLayers) {
        const bool one_launch = step_uses_one_launch(c);  // asked before the append moves the lengths
        int rc = step_append(c, k, v, s);
        if (rc) return rc;
        if (one_launch) return do_decode_step(c, 0, c->layers, q, out, s, true);
        return step_decode(c, 0, c->layers, q, out, s, false);
    }
    for (int l = 0; l < c->layers; ++l) {
        int rc = do_append(c, l, static_cast<const __nv_bfloat16*>(k) + l * kv_layer,
                           static_cast<const __nv_bfloat16*>(v) + l * kv_layer, 1, s);
        if (rc) return rc;
        rc = do_decode(c, l, static_cast<const __nv_bfloat16*>(q) + l * q_layer,
                       static_cast<uint8_t*>(out) + l * q_layer * (c->out_bf16 ? 2 : 4), s);
        if (rc) return rc;
    }
    return RLKV_OK;
}

int rlkv_step_host(rlkv_cache* c, const void* k_host, const void* v_host, const void* q_host, void* out_host,
                   void* stream)
{
    if (!c || !k_host || !v_host || !q_host || !out_host) return RLKV_EINVAL;
    for (int l = 0; l < c->layers; ++l)
        if (c->len[l] >= c->max_len) return RLKV_EFULL;
    DeviceGuard g(c->device);
    if (!g.ok) return RLKV_ECUDA;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t kv_bytes = (size_t)c->layers * c->batch * c->kv_heads * c->head_dim * 2;
    const size_t q_bytes = (size_t)c->layers * c->batch * c->q_heads * c->head_dim * 2;
    if (c->fp8) {  // in, step, out, all on the caller's stream
        uint8_t* dk = c->fp8_staging;
        uint8_t* dv = dk + align_up(kv_bytes, 256);
        uint8_t* dq = dv + align_up(kv_bytes, 256);
        uint8_t* dout = dq + align_up(q_bytes, 256);
        RLKV_CUDA(cudaMemcpyAsync(dk, k_host, kv_bytes, cudaMemcpyHostToDevice, s));
        RLKV_CUDA(cudaMemcpyAsync(dv, v_host, kv_bytes, cudaMemcpyHostToDevice, s));
        RLKV_CUDA(cudaMemcpyAsync(dq, q_host, q_bytes, cudaMemcpyHostToDevice, s));
        const int rc = fp8_step(c, dk, dv, dq, dout, stream);
        if (rc) return rc;
        RLKV_CUDA(cudaMemcpyAsync(out_host, dout, q_bytes * (c->out_bf16 ? 1 : 2), cudaMemcpyDeviceToHost, s));
        return RLKV_OK;
    }
    const int chunks = c->layers >= 8 ? 2 : 1;
    if (chunks == 1 || c->layers > kMaxStepLayers) {
        uint8_t* dk = c->dev_base + c->lay.off_k;
        uint8_t* dv = c->dev_base + c->lay.off_v;
        uint8_t* dq = c->dev_base + c->lay.off_q;
        uint8_t* dout = c->dev_base + c->lay.off_out;
        RLKV_CUDA(cudaMemcpyAsync(dk, k_host, kv_bytes, cudaMemcpyHostToDevice, s));
        RLKV_CUDA(cudaMemcpyAsync(dv, v_host, kv_bytes, cudaMemcpyHostToDevice, s));
        RLKV_CUDA(cudaMemcpyAsync(dq, q_host, q_bytes, cudaMemcpyHostToDevice, s));
        int rc = rlkv_step(c, dk, dv, dq, dout, stream);
        if (rc) return rc;
        RLKV_CUDA(cudaMemcpyAsync(out_host, dout, q_bytes * (c->out_bf16 ? 1 : 2), cudaMemcpyDeviceToHost, s));
        return RLKV_OK;
    }
    // Inputs come in on one side stream, results go out on another, both beside the kernels on the
    // caller's stream.  The input staging area exists twice and calls alternate between the copies,
    // so this call's inputs can be copied in while the kernels of the call before still read theirs.
    // The layers go in two chunks, the last eighth apart: little is left to copy out after the last
    // kernel, and the results of the first chunk leave while the second is computed.  (Every further
    // chunk costs a launch, about 25 us measured; four chunks -- a short first one for the inputs as
    // well -- measured 50 us slower per step once consecutive calls overlap, since the inputs of a call
    // then arrive during the call before anyway.)
    const int p = (int)(c->host_steps++ & 1);
    const size_t in_bytes = c->lay.off_out - c->lay.off_k;          // k, v, q of one copy
    uint8_t* dk = c->dev_base + c->lay.off_k + (p ? c->lay.off_in2 - c->lay.off_k : 0);
    uint8_t* dv = dk + (c->lay.off_v - c->lay.off_k);
    uint8_t* dq = dk + (c->lay.off_q - c->lay.off_k);
    uint8_t* dout = c->dev_base + c->lay.off_out;
    (void)in_bytes;
    const size_t q_layer = q_bytes / c->layers;
    const int L = c->layers, tail = L / 8 > 0 ? L / 8 : 1;
    const int bounds[3] = {0, L - tail, L};
    // inputs: this copy of the staging area was last read by the kernels of the call before last
    RLKV_CUDA(cudaStreamWaitEvent(c->in_stream, c->ev_step[p], 0));
    RLKV_CUDA(cudaMemcpyAsync(dk, k_host, kv_bytes, cudaMemcpyHostToDevice, c->in_stream));
    RLKV_CUDA(cudaMemcpyAsync(dv, v_host, kv_bytes, cudaMemcpyHostToDevice, c->in_stream));
    for (int i = 0; i < chunks; ++i) {
        const size_t o = q_layer * bounds[i], n = q_layer * (bounds[i + 1] - bounds[i]);
        RLKV_CUDA(cudaMemcpyAsync(dq + o, static_cast<const uint8_t*>(q_host) + o, n, cudaMemcpyHostToDevice,
                                  c->in_stream));
        RLKV_CUDA(cudaEventRecord(c->ev_in[i], c->in_stream));
    }
    // kernels: per chunk of layers one attention launch over all its layers where the step allows it,
    // else one launch per layer
    RLKV_CUDA(cudaStreamWaitEvent(s, c->ev_in[0], 0));
    const bool one_launch = step_uses_one_launch(c);
    int rc = step_append(c, dk, dv, s);
    if (rc) return rc;
    for (int i = 0; i < chunks; ++i) {
        if (i > 0) RLKV_CUDA(cudaStreamWaitEvent(s, c->ev_in[i], 0));
        rc = one_launch ? do_decode_step(c, bounds[i], bounds[i + 1], dq, dout, s, i == 0)
                        : step_decode(c, bounds[i], bounds[i + 1], dq, dout, s, i > 0);
        if (rc) return rc;
        RLKV_CUDA(cudaEventRecord(c->ev_out[i], s));
        // results of the chunk
        const size_t ob = c->out_bf16 ? 1 : 2;  // bytes of a result element / bytes of a query element
        const size_t o = ob * q_layer * bounds[i], n = ob * q_layer * (bounds[i + 1] - bounds[i]);
        RLKV_CUDA(cudaStreamWaitEvent(c->out_stream, c->ev_out[i], 0));
        RLKV_CUDA(cudaMemcpyAsync(static_cast<uint8_t*>(out_host) + o, dout + o, n, cudaMemcpyDeviceToHost,
                                  c->out_stream));
    }
    RLKV_CUDA(cudaEventRecord(c->ev_step[p], s));             // this call's kernels are done with their inputs
    RLKV_CUDA(cudaEventRecord(c->ev_done, c->out_stream));   // whoever waits for s also waits for the results
    RLKV_CUDA(cudaStreamWaitEvent(s, c->ev_done, 0));
    return RLKV_OK;
}

int rlkv_length(const rlkv_cache* c, int layer, int* len_out)
{
    if (!valid_layer(c, layer) || !len_out) return RLKV_EINVAL;
    *len_out = c->len[layer];
    return RLKV_OK;
}

int rlkv_step_bytes(const rlkv_cache* c, int layer, uint64_t* kv_bytes_out)
{
    if (!valid_layer(c, layer) || !kv_bytes_out) return RLKV_EINVAL;
    if (c->fp8) return rlkv_paged_step_bytes(c->fp8, layer, c->fp8_slots.data(), c->batch, kv_bytes_out);
    const uint64_t n = (uint64_t)c->len[layer], cap = (uint64_t)c->sink + c->window;
    const uint64_t row_pair = (uint64_t)c->head_dim * 2 * 2;  // one K row + one V row
    const uint64_t rows = (uint64_t)c->lay.n_full[layer] * n + (uint64_t)c->lay.n_comp[layer] * (n < cap ? n : cap);
    *kv_bytes_out = (uint64_t)c->batch * rows * row_pair;
    return RLKV_OK;
}

int rlkv_debug_export_head(rlkv_cache* c, int layer, int b, int h, void* k_host, void* v_host, int* rows_out,
                           int32_t* token_of_slot)
{
    if (!valid_layer(c, layer) || b < 0 || b >= c->batch || h < 0 || h >= c->kv_heads || !k_host || !v_host ||
        !rows_out || !token_of_slot)
        return RLKV_EINVAL;
    DeviceGuard g(c->device);
    if (!g.ok) return RLKV_ECUDA;
    if (c->fp8) return fp8_export(c, layer, b, h, k_host, v_host, rows_out, token_of_slot);
    RLKV_CUDA(cudaDeviceSynchronize());
    const int slot = c->slot_of_head[layer * c->kv_heads + h];
    const int n = c->len[layer];
    long long krow;
    int rows, stride;
    if (slot >= 0) {
        rows = c->max_len;
        stride = c->lay.rows_full;
        krow = c->lay.full_row0[layer] + (long long)(b * c->lay.n_full[layer] + slot) * 2 * stride;
        for (int s = 0; s < rows; ++s) token_of_slot[s] = s < n ? s : -1;
    } else {
        rows = c->sink + c->window;
        stride = c->lay.rows_comp;
        krow = c->lay.comp_row0[layer] + (long long)(b * c->lay.n_comp[layer] + (-slot - 1)) * 2 * stride;
        for (int s = 0; s < rows; ++s) {
            int tok = -1;
            if (s < c->sink) {
                if (s < n) tok = s;
            } else if (n > c->sink) {
                // newest token t < n with sink + (t - sink) % window == s
                const int newest = n - 1, r = s - c->sink;
                const int back = (((newest - c->sink) % c->window) - r + c->window) % c->window;
                if (newest - back >= c->sink) tok = newest - back;
            }
            token_of_slot[s] = tok;
        }
    }
    const size_t bytes = (size_t)rows * c->head_dim * 2;
    const uint8_t* pool = c->dev_base + c->lay.off_pool;
    RLKV_CUDA(cudaMemcpy(k_host, pool + (size_t)krow * c->head_dim * 2, bytes, cudaMemcpyDeviceToHost));
    RLKV_CUDA(cudaMemcpy(v_host, pool + (size_t)(krow + stride) * c->head_dim * 2, bytes, cudaMemcpyDeviceToHost));
    *rows_out = rows;
    return RLKV_OK;
}

int rlkv_kernel_status(rlkv_cache* c, int* status_out)
{
    if (!c || !status_out) return RLKV_EINVAL;
    if (c->fp8) return rlkv_paged_kernel_status(c->fp8, status_out);
    DeviceGuard g(c->device);
    if (!g.ok) return RLKV_ECUDA;
    RLKV_CUDA(cudaDeviceSynchronize());
    RLKV_CUDA(cudaMemcpy(status_out, c->dev_base + c->lay.off_status, sizeof(int), cudaMemcpyDeviceToHost));
    return *status_out == 0 ? RLKV_OK : RLKV_EKERNEL;
}

int rlkv_debug_trace(rlkv_cache* c, int enable, unsigned long long* words_host, int* ctas_out)
{
    if (!c || c->fp8) return RLKV_EINVAL;
    if (words_host) {
        if (!ctas_out) return RLKV_EINVAL;
        DeviceGuard g(c->device);
        if (!g.ok) return RLKV_ECUDA;
        RLKV_CUDA(cudaDeviceSynchronize());
        RLKV_CUDA(cudaMemcpy(words_host, c->dev_base + c->lay.off_trace,
                             (size_t)c->lay.max_grid * kTraceWords * sizeof(unsigned long long),
                             cudaMemcpyDeviceToHost));
        *ctas_out = c->lay.max_grid;
    }
    c->trace_on = enable ? 1 : 0;
    return RLKV_OK;
}

int rlkv_debug_schedule(int full_units, int tiles_full, int comp_units, int tiles_comp, int ctas, int item_tiles,
                        int whole_step, int* n_items_out, int* n_slots_out, int* starts_out, int* tile_map_out, int cap)
{
    if (full_units < 0 || comp_units < 0 || full_units + comp_units < 1 || tiles_full < 1 || tiles_comp < 1 ||
        ctas < 1 || item_tiles < 1 || !n_items_out || !n_slots_out)
        return RLKV_EINVAL;
    if ((long long)full_units * tiles_full + (long long)comp_units * tiles_comp >= (1ll << 31)) return RLKV_EINVAL;
    const Schedule sc = whole_step ? step_schedule(full_units, tiles_full, comp_units, tiles_comp, ctas, item_tiles, true, -1, whole_step == 2)
                                   : make_schedule(full_units, tiles_full, comp_units, tiles_comp, ctas, item_tiles);
    *n_items_out = sc.n_items;
    *n_slots_out = sc.n_slots;
    if (!whole_step && max_slots(full_units, tiles_full, comp_units, tiles_comp, ctas, item_tiles) < sc.n_slots)
        return RLKV_EKERNEL;
    if (starts_out) {
        if (cap < sc.n_items + 1) return RLKV_ENOMEM;
        for (int k = 0; k <= sc.n_items; ++k) starts_out[k] = item_start(sc, k);
        for (int k = 0; k < sc.n_items; ++k)  // the inverse map must agree with the starts
            for (int x = starts_out[k]; x < starts_out[k + 1]; ++x)
                if (item_of_tile(sc, x) != k) return RLKV_EKERNEL;
    }
    if (tile_map_out) {
        if (cap < sc.T) return RLKV_ENOMEM;
        for (int x = 0; x < sc.T; ++x) {
            const TilePos p = tile_pos(sc, x);
            tile_map_out[4 * x + 0] = p.uid;
            tile_map_out[4 * x + 1] = p.tile;
            tile_map_out[4 * x + 2] = p.run;
            tile_map_out[4 * x + 3] = partial_slot(sc, p.band, item_of_tile(sc, x), p.uid);
            // the per-unit list of partial records must contain the record of every tile's segment
            int slot = 0, count = 0;
            unit_partials(sc, p.uid, p.band < 0 ? 0 : p.band, slot, count);
            if (tile_map_out[4 * x + 3] < slot || tile_map_out[4 * x + 3] >= slot + count) return RLKV_EKERNEL;
            if (tile_map_out[4 * x + 3] >= sc.n_slots) return RLKV_EKERNEL;
        }
    }
    return RLKV_OK;
}

int rlkv_debug_claim_order(int full_units, int tiles_full, int comp_units, int tiles_comp, int ctas, int item_tiles,
                           int whole_step, int* order_out, int cap)
{
    if (full_units < 0 || comp_units < 0 || full_units + comp_units < 1 || tiles_full < 1 || tiles_comp < 1 ||
        ctas < 1 || item_tiles < 1 || !order_out)
        return RLKV_EINVAL;
    if ((long long)full_units * tiles_full + (long long)comp_units * tiles_comp >= (1ll << 31)) return RLKV_EINVAL;
    const Schedule sc = whole_step ? step_schedule(full_units, tiles_full, comp_units, tiles_comp, ctas, item_tiles, true, -1, whole_step == 2)
                                   : make_schedule(full_units, tiles_full, comp_units, tiles_comp, ctas, item_tiles);
    if (cap < sc.n_items) return RLKV_ENOMEM;
    for (int k = 0; k < sc.n_items; ++k) order_out[k] = claim_to_item(sc, k);
    return RLKV_OK;
}

int rlkv_debug_step_plan(int n_launches, int follows_append, int* overlap_out, int* dep_wait_out, int* scratch_copy_out)
{
    if (n_launches < 1 || !overlap_out || !dep_wait_out || !scratch_copy_out) return RLKV_EINVAL;
    for (int l = 0; l < n_launches; ++l) {
        const StepLaunchMode m = step_launch_mode(l == 0, follows_append != 0);
        overlap_out[l] = m.overlap ? 1 : 0;
        dep_wait_out[l] = m.dep_wait;
        scratch_copy_out[l] = l & 1;
    }
    return RLKV_OK;
}

int rlkv_launch_count(const rlkv_cache* c, uint64_t* launches_out)
{
    if (!c || !launches_out) return RLKV_EINVAL;
    *launches_out = c->fp8 ? paged_launch_count(c->fp8) : c->launches;
    return RLKV_OK;
}

}  // extern "C"
