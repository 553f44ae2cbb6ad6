// Host side of the paged, ragged cache of librlkv (rlkv_paged_* in include/rlkv.h): request slots
// with their own lengths, full heads in 64-token pages handed out from one free list, compressed
// heads in a constant-size ring per request slot (the serving layout of Section 4.3 of the paper:
// a paged pool for the full heads beside a fixed-size pool for the compressed ones).
//
// Device buffer (sections 1024-byte aligned):
//   pool        rows of head_dim bf16.  Per layer: the full-head region
//               [n_full(layer)][n_pages][K|V][64][D] -- page p of a sequence is page p of every full
//               head of every layer -- then the compressed-head region
//               [max_seqs][n_comp(layer)][K|V][rows_comp][D]
//   pool8       only with 8-bit storage (rlkv_paged_create_fp8; the 16-bit pool is then empty): pages of
//               16 KB (K codes [64 rows][128], then V codes transposed [128][64 rows]); per layer the
//               full heads' pages [n_full(layer)][n_pages], then the rings
//               [max_seqs][n_comp(layer)][rows_comp / 64]
//   scales      float 1/k_scale, 1/v_scale, k_scale, v_scale, each [layers][kv_heads] (8-bit pages only)
//   tables      int32 slot_of_head[layers][kv_heads]
//   page table  int32 [max_seqs][table_stride]   (written by the append kernels)
//   layer desc  LayerDesc[layers]  (where each layer's regions start; for the step's append launch)
//   tickets     int32 [2][kMaxPagedBatch * kv_heads]
//   status      int32 kernel status word, then two work-claim counters
//   partials    float [2][max_slots][partial_floats]
//               (tickets, counters and partials exist twice: the overlapped launches of
//               rlkv_paged_step alternate between the halves)
// Lengths, the page table's mirror and the free list live on the host.
#include <stdlib.h>
#include <string.h>

#include <new>
#include <vector>

#include "rlkv_host.cuh"

using namespace rlkv;

struct rlkv_paged {
    int layers, kv_heads, q_heads, head_dim, max_seqs, n_pages, table_stride, sink, window;
    int max_seq_len;              // most tokens a sequence may hold (the page table is laid out for a few more)
    int device, sm_count, stages, groups, item_tiles;
    int rows_comp, max_batch, max_items, max_grid;
    int out_bf16;
    int step_mode;                // rlkv_paged_step: 0 chooses, 1 one decode launch per layer, 2 one for the whole step
    bool step_in_one_launch;      // the shape allows one decode launch for a whole step
    long long step_slots;         // partial records the scratch holds when both copies are used as one
    int fp8;                      // K/V rows (pages and rings) are held as E4M3 codes
    std::vector<float> k_scale, v_scale;  // [layers*kv_heads]
    std::vector<long long> page0_8, ring0_8;  // first full-head page / first ring page of each layer in the 8-bit pool
    long long pages8;                      // pages of the 8-bit pool
    size_t off_pool8, off_scales;
    CUtensorMap map_k;  // the 8-bit pool as rows of 128 bytes, one page per box
    long long pool_rows;
    std::vector<uint8_t> is_full;
    std::vector<int> slot_of_head, head_of_slot;  // [layers*kv_heads]
    std::vector<int> n_full, n_comp;
    std::vector<long long> full_row0, comp_row0;
    std::vector<int> len;         // [layers][max_seqs]
    std::vector<int> table;       // [max_seqs][table_stride], -1 = no page
    std::vector<int> free_pages;  // stack of physical pages
    std::vector<uint8_t> open;    // [max_seqs]
    size_t off_pool, off_tables, off_head_table, off_layer_desc, off_page_table, off_tickets, off_status, off_partials, total;
    unsigned int claims[2];
    uint8_t* dev_base;
    bool owns_buffer;
    CUtensorMap tmap;
    uint64_t launches;
};

namespace {

constexpr int kPagedItemTiles = 8;       // smallest work item of a launch on its own
constexpr int kPagedItemTilesStep = 32;  // and of the overlapped launches of rlkv_paged_step
constexpr int kPagedMaxFanIn = 32;

int check_paged_shape(int layers, int kv_heads, int q_heads, int head_dim, int max_seqs, int n_pages,
                      int max_seq_len, const uint8_t* mask, int sink, int window)
{
    if (!mask || layers < 1 || kv_heads < 1 || kv_heads > kMaxKvHeads || q_heads < 1 || max_seqs < 1 ||
        max_seqs > 65535 || n_pages < 1 || max_seq_len < 1)
        return RLKV_EINVAL;
    if (q_heads % kv_heads != 0 || q_heads / kv_heads > kMaxGroup) return RLKV_EINVAL;
    if (head_dim != 64 && head_dim != 128) return RLKV_EINVAL;
    if (sink < 0 || window < 1 || (long long)sink + window > (1 << 24)) return RLKV_EINVAL;
    if (max_seq_len > kMaxSeqPages * kTile) return RLKV_EINVAL;
    return RLKV_OK;
}

// Fills the shape-dependent fields of `p` (no device work).
int make_paged_layout(rlkv_paged& p, const uint8_t* mask, int max_seq_len)
{
    p.table_stride = (int)align_up((size_t)(max_seq_len + kTile - 1) / kTile, 4);
    p.rows_comp = (int)align_up((size_t)p.sink + p.window, kTile);
    p.max_batch = p.max_seqs < kMaxPagedBatch ? p.max_seqs : kMaxPagedBatch;
    p.max_grid = 2 * kMaxGridSms;
    p.is_full.assign(mask, mask + (size_t)p.layers * p.kv_heads);
    p.slot_of_head.assign((size_t)p.layers * p.kv_heads, 0);
    p.head_of_slot.assign((size_t)p.layers * p.kv_heads, 0);
    p.n_full.assign(p.layers, 0);
    p.n_comp.assign(p.layers, 0);
    p.full_row0.assign(p.layers, 0);
    p.comp_row0.assign(p.layers, 0);
    p.page0_8.assign(p.layers, 0);
    p.ring0_8.assign(p.layers, 0);
    p.pages8 = 0;
    long long row = 0, most = 0;
    for (int l = 0; l < p.layers; ++l) {
        int nf = 0, nc = 0;
        for (int h = 0; h < p.kv_heads; ++h)
            if (mask[l * p.kv_heads + h]) p.slot_of_head[l * p.kv_heads + h] = nf++;
            else p.slot_of_head[l * p.kv_heads + h] = -(++nc);
        for (int h = 0; h < p.kv_heads; ++h) {
            const int s = p.slot_of_head[l * p.kv_heads + h];
            p.head_of_slot[l * p.kv_heads + (s >= 0 ? s : nf + (-s - 1))] = h;
        }
        p.n_full[l] = nf;
        p.n_comp[l] = nc;
        p.full_row0[l] = row;
        if (p.fp8) {
            p.page0_8[l] = p.pages8;
            p.pages8 += (long long)nf * p.n_pages;
            p.ring0_8[l] = p.pages8;
            p.pages8 += (long long)p.max_seqs * nc * (p.rows_comp / kTile);
            p.comp_row0[l] = row;
        } else {
            row += (long long)nf * p.n_pages * 2 * kTile;
            p.comp_row0[l] = row;
            row += (long long)p.max_seqs * nc * 2 * p.rows_comp;
        }
        const long long t = (long long)p.max_batch * ((long long)nf * p.table_stride + (long long)nc * (p.rows_comp / kTile));
        if (t >= (1ll << 31)) return RLKV_EINVAL;
        const long long m = most_slots(p.max_batch * nf, p.table_stride, p.max_batch * nc, p.rows_comp / kTile, p.max_grid);
        if (m > most) most = m;
    }
    if (row >= (1ll << 31) || most >= (1ll << 31)) return RLKV_EINVAL;  // TMA row coordinates are 32-bit
    if (p.pages8 * 128 >= (1ll << 31)) return RLKV_EINVAL;              // a page is 128 rows of the 8-bit map
    p.pool_rows = row;
    // A whole step in one launch uses both copies of the scratch as one.  Sized for max_batch sequences
    // of max_seq_len tokens where that is modest (at most 64 MB more per copy); a step that needs more
    // records than there are runs as one launch per layer.
    p.step_in_one_launch = p.layers <= kMaxStepLayers && p.layers * p.kv_heads <= kMaxStepHeads;
    if (p.step_in_one_launch) {
        long long U = 0, Uc = 0;
        for (int l = 0; l < p.layers; ++l) {
            U += (long long)p.max_batch * p.n_full[l];
            Uc += (long long)p.max_batch * p.n_comp[l];
        }
        const long long T = U * p.table_stride + Uc * (p.rows_comp / kTile);
        const long long small = (long long)p.max_grid * kDefaultItemTiles / kMinItemTiles + 1;
        const long long large = T / kDefaultItemTiles + 1;
        long long fused = 2ll * p.max_grid + 2 * U + Uc + (small > large ? small : large) + 8;
        const long long cap = most + (64ll << 20) / ((long long)partial_floats(p.head_dim, p.q_heads / p.kv_heads) * 4);
        if ((fused + 1) / 2 > cap) fused = 2 * cap;
        if ((fused + 1) / 2 > most) most = (fused + 1) / 2;
    }
    p.max_items = (int)most;
    p.step_slots = 2ll * most;
    size_t off = 0;
    p.off_pool = off;
    off = align_up(off + (size_t)row * p.head_dim * 2, 1024);
    p.off_pool8 = off;
    off = align_up(off + (size_t)p.pages8 * 2 * kTile * 128, 1024);
    p.off_scales = off;
    off = align_up(off + (p.fp8 ? (size_t)4 * p.layers * p.kv_heads * sizeof(float) : 0), 1024);
    p.off_tables = off;
    off = align_up(off + (size_t)p.layers * p.kv_heads * sizeof(int), 1024);
    p.off_head_table = off;  // head_of_slot, for a whole-step launch
    off = align_up(off + (size_t)p.layers * p.kv_heads * sizeof(int), 1024);
    p.off_layer_desc = off;
    off = align_up(off + (size_t)p.layers * sizeof(LayerDesc), 1024);
    p.off_page_table = off;
    off = align_up(off + (size_t)p.max_seqs * p.table_stride * sizeof(int), 1024);
    p.off_tickets = off;
    {   // two copies of one ticket per unit of a layer; a whole step needs one per unit of every layer
        const size_t per_layer = (size_t)2 * kMaxPagedBatch * p.kv_heads, whole = (size_t)p.layers * p.max_batch * p.kv_heads;
        off = align_up(off + (per_layer > whole ? per_layer : whole) * sizeof(int), 1024);
    }
    p.off_status = off;
    off = align_up(off + 64, 1024);
    p.off_partials = off;
    off = align_up(off + (size_t)2 * p.max_items * partial_floats(p.head_dim, p.q_heads / p.kv_heads) * sizeof(float), 1024);
    p.total = off;
    return RLKV_OK;
}

template <typename T>
T* dev_at(const rlkv_paged* p, size_t off) { return reinterpret_cast<T*>(p->dev_base + off); }

bool valid_layer(const rlkv_paged* p, int layer) { return p && layer >= 0 && layer < p->layers; }
bool valid_slot(const rlkv_paged* p, int slot) { return slot >= 0 && slot < p->max_seqs && p->open[slot]; }

// The request slots of a call: all open, no slot twice.
int check_slots(const rlkv_paged* p, const int* slots, int n)
{
    if (!slots || n < 1 || n > p->max_batch) return RLKV_EINVAL;
    std::vector<uint8_t> seen(p->max_seqs, 0);
    for (int i = 0; i < n; ++i) {
        if (!valid_slot(p, slots[i]) || seen[slots[i]]) return RLKV_EINVAL;
        seen[slots[i]] = 1;
    }
    return RLKV_OK;
}

int* len_of(rlkv_paged* p, int layer) { return p->len.data() + (size_t)layer * p->max_seqs; }
const int* len_of(const rlkv_paged* p, int layer) { return p->len.data() + (size_t)layer * p->max_seqs; }

void fill_append_args(rlkv_paged* p, int layer, const void* k, const void* v, PagedAppendArgs& a)
{
    a.pool = dev_at<__nv_bfloat16>(p, p->off_pool);
    a.page_table = dev_at<int>(p, p->off_page_table);
    a.full_row0 = p->full_row0[layer];
    a.comp_row0 = p->comp_row0[layer];
    a.slot_of_head = dev_at<int>(p, p->off_tables) + (size_t)layer * p->kv_heads;
    a.k = static_cast<const __nv_bfloat16*>(k);
    a.v = static_cast<const __nv_bfloat16*>(v);
    a.n_full = p->n_full[layer];
    a.n_comp = p->n_comp[layer];
    a.rows_comp = p->rows_comp;
    a.n_pages = p->n_pages;
    a.table_stride = p->table_stride;
    a.kv_heads = p->kv_heads;
    a.head_dim = p->head_dim;
    a.sink = p->sink;
    a.window = p->window;
    a.n_layers = 1;
    a.layers = nullptr;
    a.entry_stride = (long long)p->kv_heads * p->head_dim;
    a.pool8 = p->fp8 ? p->dev_base + p->off_pool8 : nullptr;
    a.k_inv = dev_at<float>(p, p->off_scales) + (size_t)layer * p->kv_heads;
    a.v_inv = a.k_inv + (size_t)p->layers * p->kv_heads;
    a.page0_8 = p->page0_8[layer];
    a.ring0_8 = p->ring0_8[layer];
    a.ring_tiles = p->rows_comp / kTile;
}

}  // namespace

extern "C" {

static int paged_size(int layers, int kv_heads, int q_heads, int head_dim, int max_seqs, int n_pages, int max_seq_len,
                      const uint8_t* head_is_full, int sink, int window, int fp8, size_t* bytes_out)
{
    if (!bytes_out) return RLKV_EINVAL;
    int rc = check_paged_shape(layers, kv_heads, q_heads, head_dim, max_seqs, n_pages, max_seq_len, head_is_full, sink, window);
    if (rc) return rc;
    if (fp8 && head_dim != 128) return RLKV_EINVAL;
    rlkv_paged p{};
    p.layers = layers; p.kv_heads = kv_heads; p.q_heads = q_heads; p.head_dim = head_dim;
    p.max_seqs = max_seqs; p.n_pages = n_pages; p.sink = sink; p.window = window; p.fp8 = fp8;
    rc = make_paged_layout(p, head_is_full, max_seq_len);
    if (rc) return rc;
    *bytes_out = p.total;
    return RLKV_OK;
}

int rlkv_paged_size(int layers, int kv_heads, int q_heads, int head_dim, int max_seqs, int n_pages, int max_seq_len,
                    const uint8_t* head_is_full, int sink, int window, size_t* bytes_out)
{
    return paged_size(layers, kv_heads, q_heads, head_dim, max_seqs, n_pages, max_seq_len, head_is_full, sink, window, 0,
                      bytes_out);
}

int rlkv_paged_size_fp8(int layers, int kv_heads, int q_heads, int head_dim, int max_seqs, int n_pages, int max_seq_len,
                        const uint8_t* head_is_full, int sink, int window, size_t* bytes_out)
{
    return paged_size(layers, kv_heads, q_heads, head_dim, max_seqs, n_pages, max_seq_len, head_is_full, sink, window, 1,
                      bytes_out);
}

static int paged_create(rlkv_paged** out, int layers, int kv_heads, int q_heads, int head_dim, int max_seqs, int n_pages,
                        int max_seq_len, const uint8_t* head_is_full, int sink, int window, const float* k_scale,
                        const float* v_scale, void* device_buf, size_t device_buf_bytes)
{
    if (!out) return RLKV_EINVAL;
    *out = nullptr;
    int rc = check_paged_shape(layers, kv_heads, q_heads, head_dim, max_seqs, n_pages, max_seq_len, head_is_full, sink, window);
    if (rc) return rc;
    const int fp8 = k_scale != nullptr;
    if (fp8) {
        if (!v_scale || head_dim != 128) return RLKV_EINVAL;
        for (int i = 0; i < layers * kv_heads; ++i)
            if (!(k_scale[i] > 0.f) || !(v_scale[i] > 0.f) || k_scale[i] > 3.0e38f || v_scale[i] > 3.0e38f) return RLKV_EINVAL;
    }
    rlkv_paged* p = new (std::nothrow) rlkv_paged();
    if (!p) return RLKV_ENOMEM;
    p->layers = layers; p->kv_heads = kv_heads; p->q_heads = q_heads; p->head_dim = head_dim;
    p->max_seqs = max_seqs; p->n_pages = n_pages; p->sink = sink; p->window = window; p->max_seq_len = max_seq_len;
    p->claims[0] = p->claims[1] = 0; p->launches = 0; p->dev_base = nullptr; p->owns_buffer = false; p->out_bf16 = 0;
    p->step_mode = 0;
    p->fp8 = fp8;
    if (fp8) {
        p->k_scale.assign(k_scale, k_scale + (size_t)layers * kv_heads);
        p->v_scale.assign(v_scale, v_scale + (size_t)layers * kv_heads);
    }
    rc = make_paged_layout(*p, head_is_full, max_seq_len);
    if (rc) { delete p; return rc; }
    p->len.assign((size_t)layers * max_seqs, 0);
    p->table.assign((size_t)max_seqs * p->table_stride, -1);
    p->open.assign(max_seqs, 0);
    p->free_pages.resize(n_pages);
    for (int i = 0; i < n_pages; ++i) p->free_pages[i] = n_pages - 1 - i;  // page 0 is handed out first
    cudaError_t e = cudaGetDevice(&p->device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&p->sm_count, cudaDevAttrMultiProcessorCount, p->device);
    if (e != cudaSuccess) { delete p; return cuda_fail(e, "device query"); }
    p->groups = 2;
    p->item_tiles = kPagedItemTiles;
    p->stages = max_stages(head_dim, q_heads / kv_heads, p->groups, 1, fp8 ? kModePagedFp8 : kModePaged);
    if (p->stages < 2) { delete p; return RLKV_EINVAL; }
    if (device_buf) {
        if ((reinterpret_cast<uintptr_t>(device_buf) & 1023u) != 0 || device_buf_bytes < p->total) { delete p; return RLKV_ENOMEM; }
        p->dev_base = static_cast<uint8_t*>(device_buf);
    } else {
        void* mem = nullptr;
        e = cudaMalloc(&mem, p->total);
        if (e != cudaSuccess) { cudaGetLastError(); delete p; return RLKV_ENOMEM; }
        p->dev_base = static_cast<uint8_t*>(mem);
        p->owns_buffer = true;
    }
    auto fail = [&](int code) {
        if (p->owns_buffer) cudaFree(p->dev_base);
        delete p;
        return code;
    };
    // pools zero-filled (rows never written stay finite), tickets / status / counter start at zero
    e = cudaMemset(p->dev_base + p->off_pool, 0, (size_t)p->pool_rows * head_dim * 2);
    if (e == cudaSuccess && fp8) e = cudaMemset(p->dev_base + p->off_pool8, 0, (size_t)p->pages8 * 2 * kTile * 128);
    if (e == cudaSuccess && fp8) {
        // the kernels multiply by 1 / scale: one IEEE division per head, here
        std::vector<float> inv((size_t)4 * layers * kv_heads);  // then the scales themselves, for a whole-step launch
        for (int i = 0; i < layers * kv_heads; ++i) {
            inv[i] = 1.0f / k_scale[i];
            inv[(size_t)layers * kv_heads + i] = 1.0f / v_scale[i];
            inv[(size_t)2 * layers * kv_heads + i] = k_scale[i];
            inv[(size_t)3 * layers * kv_heads + i] = v_scale[i];
        }
        e = cudaMemcpy(p->dev_base + p->off_scales, inv.data(), inv.size() * sizeof(float), cudaMemcpyHostToDevice);
    }
    if (e == cudaSuccess) e = cudaMemset(p->dev_base + p->off_page_table, 0, p->off_partials - p->off_page_table);
    if (e == cudaSuccess)
        e = cudaMemcpy(p->dev_base + p->off_tables, p->slot_of_head.data(), p->slot_of_head.size() * sizeof(int),
                       cudaMemcpyHostToDevice);
    if (e == cudaSuccess)
        e = cudaMemcpy(p->dev_base + p->off_head_table, p->head_of_slot.data(), p->head_of_slot.size() * sizeof(int),
                       cudaMemcpyHostToDevice);
    if (e == cudaSuccess) {
        std::vector<LayerDesc> desc(layers);
        for (int l = 0; l < layers; ++l) desc[l] = LayerDesc{p->full_row0[l], p->comp_row0[l], p->n_full[l], p->n_comp[l], p->page0_8[l], p->ring0_8[l]};
        e = cudaMemcpy(p->dev_base + p->off_layer_desc, desc.data(), desc.size() * sizeof(LayerDesc), cudaMemcpyHostToDevice);
    }
    if (e == cudaSuccess) e = prepare_decode_kernels(head_dim);
    if (e != cudaSuccess) return fail(cuda_fail(e, "rlkv_paged_create"));
    // (a pool without rows -- every head full and in 8-bit pages -- still gets a one-row map: it is never used)
    rc = encode_pool_tensor_map(&p->tmap, p->dev_base + p->off_pool, p->pool_rows > 0 ? p->pool_rows : 1, head_dim);
    if (rc) return fail(rc);
    if (fp8 && p->pages8 > 0) {
        rc = encode_byte_rows_tensor_map(&p->map_k, p->dev_base + p->off_pool8, 128, p->pages8 * 128, 2 * kTile);
        if (rc) return fail(rc);
    }
    *out = p;
    return RLKV_OK;
}

int rlkv_paged_create(rlkv_paged** out, int layers, int kv_heads, int q_heads, int head_dim, int max_seqs, int n_pages,
                      int max_seq_len, const uint8_t* head_is_full, int sink, int window, void* device_buf,
                      size_t device_buf_bytes)
{
    return paged_create(out, layers, kv_heads, q_heads, head_dim, max_seqs, n_pages, max_seq_len, head_is_full, sink, window,
                        nullptr, nullptr, device_buf, device_buf_bytes);
}

int rlkv_paged_create_fp8(rlkv_paged** out, int layers, int kv_heads, int q_heads, int head_dim, int max_seqs, int n_pages,
                          int max_seq_len, const uint8_t* head_is_full, int sink, int window, const float* k_scale,
                          const float* v_scale, void* device_buf, size_t device_buf_bytes)
{
    if (!k_scale || !v_scale) return RLKV_EINVAL;
    return paged_create(out, layers, kv_heads, q_heads, head_dim, max_seqs, n_pages, max_seq_len, head_is_full, sink, window,
                        k_scale, v_scale, device_buf, device_buf_bytes);
}

int rlkv_paged_destroy(rlkv_paged* p)
{
    if (!p) return RLKV_EINVAL;
    DeviceGuard g(p->device);
    cudaDeviceSynchronize();
    if (p->owns_buffer) cudaFree(p->dev_base);
    delete p;
    return RLKV_OK;
}

int rlkv_paged_seq_open(rlkv_paged* p, int* slot_out)
{
    if (!p || !slot_out) return RLKV_EINVAL;
    for (int s = 0; s < p->max_seqs; ++s)
        if (!p->open[s]) {
            p->open[s] = 1;
            *slot_out = s;
            return RLKV_OK;
        }
    return RLKV_EFULL;
}

int rlkv_paged_seq_close(rlkv_paged* p, int slot)
{
    if (!p || !valid_slot(p, slot)) return RLKV_EINVAL;
    int* row = p->table.data() + (size_t)slot * p->table_stride;
    for (int i = p->table_stride - 1; i >= 0; --i)
        if (row[i] >= 0) {
            p->free_pages.push_back(row[i]);
            row[i] = -1;
        }
    for (int l = 0; l < p->layers; ++l) len_of(p, l)[slot] = 0;
    p->open[slot] = 0;
    return RLKV_OK;
}

int rlkv_paged_append(rlkv_paged* p, int layer, const int* slots, int n, const void* k, const void* v, void* stream)
{
    if (!valid_layer(p, layer) || !k || !v || !aligned16(k) || !aligned16(v)) return RLKV_EINVAL;
    int rc = check_slots(p, slots, n);
    if (rc) return rc;
    int* len = len_of(p, layer);
    // every sequence must have room and, where its token opens a page, a free page: checked before
    // anything changes
    int need = 0;
    for (int i = 0; i < n; ++i) {
        const int t = len[slots[i]];
        if (t >= p->max_seq_len) return RLKV_EFULL;
        if (p->table[(size_t)slots[i] * p->table_stride + t / kTile] < 0) ++need;
    }
    if (need > (int)p->free_pages.size()) return RLKV_EFULL;
    DeviceGuard g(p->device);
    if (!g.ok) return RLKV_ECUDA;
    PagedAppendArgs a;
    fill_append_args(p, layer, k, v, a);
    a.prefill = 0;
    a.n = n;
    a.t0 = 0;
    a.first_page = 0;
    for (int i = 0; i < n; ++i) {
        const int s = slots[i], t = len[s];
        int& entry = p->table[(size_t)s * p->table_stride + t / kTile];
        if (entry < 0) {
            entry = p->free_pages.back();
            p->free_pages.pop_back();
        }
        a.slot[i] = (unsigned short)s;
        a.t[i] = t;
        a.page[i] = entry;
    }
    RLKV_CUDA(launch_paged_append(a, static_cast<cudaStream_t>(stream)));
    for (int i = 0; i < n; ++i) len[slots[i]] += 1;
    p->launches++;
    return RLKV_OK;
}

int rlkv_paged_prefill(rlkv_paged* p, int layer, int slot, const void* k, const void* v, int n_tokens, void* stream)
{
    return rlkv::paged_prefill_strided(p, layer, slot, k, v, n_tokens, p ? (long long)p->kv_heads * p->head_dim : 0, stream);
}

}  // extern "C"

// rlkv_paged_prefill with the tokens of k and v `entry_stride` elements apart (a multiple of 8): the rows of
// one batch row inside a [tokens][batch][kv_heads][head_dim] array, for the lock-step cache kept in 8 bits.
int rlkv::paged_prefill_strided(rlkv_paged* p, int layer, int slot, const void* k, const void* v, int n_tokens,
                                long long entry_stride, void* stream)
{
    if (!valid_layer(p, layer) || !valid_slot(p, slot) || !k || !v || !aligned16(k) || !aligned16(v) || n_tokens < 1 ||
        entry_stride < (long long)p->kv_heads * p->head_dim || entry_stride % 8 != 0)
        return RLKV_EINVAL;
    int* len = len_of(p, layer);
    const int t0 = len[slot];
    if ((long long)t0 + n_tokens > p->max_seq_len) return RLKV_EFULL;
    const int first = t0 / kTile, last = (t0 + n_tokens - 1) / kTile;
    int* row = p->table.data() + (size_t)slot * p->table_stride;
    int need = 0;
    for (int i = first; i <= last; ++i)
        if (row[i] < 0) ++need;
    if (need > (int)p->free_pages.size()) return RLKV_EFULL;
    DeviceGuard g(p->device);
    if (!g.ok) return RLKV_ECUDA;
    for (int i = first; i <= last; ++i)
        if (row[i] < 0) {
            row[i] = p->free_pages.back();
            p->free_pages.pop_back();
        }
    // launches of at most kMaxAppendPages pages each: every launch equals that many single appends,
    // bit for bit, and the launches run in order, so the whole equals n_tokens single appends
    const size_t row_elems = (size_t)entry_stride;
    for (int done = 0; done < n_tokens;) {
        const int t = t0 + done;
        const int page0 = t / kTile;
        int count = n_tokens - done;
        const int room = (page0 + kMaxAppendPages) * kTile - t;  // tokens up to the end of the last page the args can name
        if (count > room) count = room;
        PagedAppendArgs a;
        fill_append_args(p, layer, static_cast<const __nv_bfloat16*>(k) + (size_t)done * row_elems,
                         static_cast<const __nv_bfloat16*>(v) + (size_t)done * row_elems, a);
        a.prefill = 1;
        a.entry_stride = entry_stride;
        a.n = count;
        a.t0 = t;
        a.first_page = page0;
        a.slot[0] = (unsigned short)slot;
        for (int i = page0; i <= (t + count - 1) / kTile; ++i) a.page[i - page0] = row[i];
        RLKV_CUDA(launch_paged_append(a, static_cast<cudaStream_t>(stream)));
        p->launches++;
        done += count;
    }
    len[slot] = t0 + n_tokens;
    return RLKV_OK;
}

uint64_t rlkv::paged_launch_count(const rlkv_paged* p) { return p ? p->launches : 0; }

extern "C" {

// One decode launch (arguments checked by the caller).  `half`: which copy of tickets, claim counter
// and partials; `overlap`, `dep_wait`: as for the lock-step cache (launch_decode, decode_kernel);
// `in_step`: the launch belongs to rlkv_paged_step (coarser items: its neighbours hide its tail).
// `whole_step`: one launch for every layer (`layer` is 0; q, out are the step's [layers][n][q_heads][head_dim]
// arrays; every listed sequence holds the same number of tokens in all layers; both scratch copies are
// used as one).  Returns RLKV_ESCRATCH, with nothing launched, if such a launch needs more partial records
// than the scratch holds: the caller then issues one launch per layer.
static int paged_decode(rlkv_paged* p, int layer, const int* slots, int n, const void* q, void* out, cudaStream_t stream,
                        int half, bool overlap, int dep_wait, bool in_step, int* grid_out, bool whole_step = false)
{
    const int* len = len_of(p, layer);
    int longest = 0;
    for (int i = 0; i < n; ++i)
        if (len[slots[i]] > longest) longest = len[slots[i]];
    const int cap = p->sink + p->window;
    DecodeArgs a;
    memset(&a, 0, sizeof a);
    a.pool = dev_at<__nv_bfloat16>(p, p->off_pool);
    a.full_row0 = p->full_row0[layer];
    a.comp_row0 = p->comp_row0[layer];
    for (int h = 0; h < p->kv_heads; ++h) a.head_of_slot[h] = (unsigned char)p->head_of_slot[(size_t)layer * p->kv_heads + h];
    a.q = static_cast<const __nv_bfloat16*>(q);
    a.out = static_cast<float*>(out);
    a.status = dev_at<int>(p, p->off_status);
    a.trace = nullptr;
    a.trace_on = 0;
    a.n_full = p->n_full[layer];
    a.n_comp = p->n_comp[layer];
    a.rows_full = 0;
    a.rows_comp = p->rows_comp;
    a.len_full = longest;
    a.len_comp = longest < cap ? longest : cap;
    a.batch = n;
    a.group = p->q_heads / p->kv_heads;
    a.q_heads = p->q_heads;
    a.scale_log2 = 1.4426950408889634f / sqrtf((float)p->head_dim);
    a.alpha = nullptr;
    a.out_bf16 = p->out_bf16;
    const int tiles_full = (a.len_full + kTile - 1) / kTile, tiles_comp = (a.len_comp + kTile - 1) / kTile;
    // the tiles that exist (the schedule also spans the ones that do not) decide the item size
    int heads_full = a.n_full, heads_comp = a.n_comp;  // per sequence, over the layers the launch serves
    if (whole_step) {
        heads_full = heads_comp = 0;
        for (int l = 0; l < p->layers; ++l) {
            heads_full += p->n_full[l];
            heads_comp += p->n_comp[l];
        }
    }
    long long real_tiles = 0;
    bool equal_lengths = true;
    for (int i = 0; i < n; ++i) {
        const int t = len[slots[i]];
        real_tiles += (long long)heads_full * ((t + kTile - 1) / kTile) + (long long)heads_comp * (((t < cap ? t : cap) + kTile - 1) / kTile);
        if (t != len[slots[0]]) equal_lengths = false;
    }
    int grid = p->sm_count;
    if (grid > p->max_grid) grid = p->max_grid;
    PagedArgs pa;
    memset(&pa, 0, sizeof pa);
    pa.step.n_layers = 1;
    if (whole_step) {
        if ((long long)n * heads_full * tiles_full + (long long)n * heads_comp * tiles_comp >= (1ll << 31)) return RLKV_ESCRATCH;
        const int most = kDefaultItemTiles * (p->fp8 ? 2 : 1);
        // equal lengths: most full units whole in one static item per CTA; else the same units, claimed one by one
        a.sched = step_schedule(n * heads_full, tiles_full, n * heads_comp, tiles_comp, grid, most, true, real_tiles, !equal_lengths);
        if (a.sched.n_slots > p->step_slots) return RLKV_ESCRATCH;
        if (grid > a.sched.n_items) grid = a.sched.n_items;
        a.n_full = a.n_comp = 0;
        a.batch = n * p->layers;
        a.partials = dev_at<float>(p, p->off_partials);
        a.tickets = dev_at<int>(p, p->off_tickets);
        a.claim_counter = dev_at<unsigned int>(p, p->off_status) + 4;
        a.claim_base = p->claims[0];
        a.dep_wait = dep_wait;
        StepArgs& st = pa.step;
        st.head_of_slot = dev_at<int>(p, p->off_head_table);
        st.n_layers = p->layers;
        st.kv_heads = p->kv_heads;
        st.batch = n;
        st.full_base[0] = st.comp_base[0] = 0;
        for (int l = 0; l < p->layers; ++l) {
            st.full_base[l + 1] = st.full_base[l] + n * p->n_full[l];
            st.comp_base[l + 1] = st.comp_base[l] + n * p->n_comp[l];
            st.full_row0[l] = (int)p->full_row0[l];
            st.comp_row0[l] = (int)p->comp_row0[l];
            pa.page0_8_of[l] = (int)p->page0_8[l];
            pa.ring0_8_of[l] = (int)p->ring0_8[l];
        }
        pa.scales = dev_at<float>(p, p->off_scales) + (size_t)2 * p->layers * p->kv_heads;
        half = 0;
    } else {
    int item_tiles = (int)(real_tiles / grid);
    // (a tile of 8-bit pages is half the bytes, so the same grain in time is twice the tiles)
    const int most = (in_step ? kPagedItemTilesStep : p->item_tiles) * (p->fp8 ? 2 : 1);
    if (item_tiles > most) item_tiles = most;
    if (item_tiles < kMinItemTiles) item_tiles = kMinItemTiles;
    a.sched = make_schedule(n * a.n_full, tiles_full, n * a.n_comp, tiles_comp, grid, item_tiles);
    // a launch too small for bands: no full unit in more than kPagedMaxFanIn pieces (their merge by one
    // CTA, not the bytes, would set the time)
    if (a.sched.R == 0 && a.n_full > 0 && tiles_full > kPagedMaxFanIn * item_tiles && (!in_step || a.sched.n_items < grid)) {
        item_tiles = (tiles_full + kPagedMaxFanIn - 1) / kPagedMaxFanIn;
        a.sched = make_schedule(n * a.n_full, tiles_full, n * a.n_comp, tiles_comp, grid, item_tiles);
    }
    if (grid > a.sched.n_items) grid = a.sched.n_items;
    if (a.sched.n_slots > p->max_items) return RLKV_ESCRATCH;  // cannot happen: the scratch is sized for it
    a.partials = dev_at<float>(p, p->off_partials) + (size_t)half * p->max_items * partial_floats(p->head_dim, a.group);
    a.tickets = dev_at<int>(p, p->off_tickets) + (size_t)half * kMaxPagedBatch * p->kv_heads;
    a.claim_counter = dev_at<unsigned int>(p, p->off_status) + 4 + half;
    a.claim_base = p->claims[half];
    a.dep_wait = dep_wait;
    }
    pa.page_table = dev_at<int>(p, p->off_page_table);
    pa.table_stride = p->table_stride;
    pa.n_pages = p->n_pages;
    pa.cap = cap;
    for (int i = 0; i < kMaxPagedBatch; ++i) {
        pa.seq_len[i] = i < n ? len[slots[i]] : 0;
        pa.seq_slot[i] = (unsigned short)(i < n ? slots[i] : 0);
    }
    pa.page0_8 = (int)p->page0_8[layer];
    pa.ring0_8 = (int)p->ring0_8[layer];
    pa.ring_tiles = p->rows_comp / kTile;
    for (int h = 0; h < kMaxKvHeads; ++h) {
        pa.k_scale[h] = p->fp8 && h < p->kv_heads ? p->k_scale[(size_t)layer * p->kv_heads + h] : 1.f;
        pa.v_scale[h] = p->fp8 && h < p->kv_heads ? p->v_scale[(size_t)layer * p->kv_heads + h] : 1.f;
    }
    if (p->fp8) {
        PagedFp8Args p8;
        p8.pa = pa;
        p8.map_k = p->map_k;
        RLKV_CUDA(launch_decode(a, &p->tmap, p->head_dim, grid, p->stages, p->groups, stream, overlap, kModePagedFp8, nullptr,
                                &p8));
    } else {
        RLKV_CUDA(launch_decode(a, &p->tmap, p->head_dim, grid, p->stages, p->groups, stream, overlap, kModePaged, &pa));
    }
    p->claims[half] += (unsigned int)a.sched.n_items;
    p->launches++;
    if (grid_out) *grid_out = grid;
    return RLKV_OK;
}

int rlkv_paged_decode_attention(rlkv_paged* p, int layer, const int* slots, int n, const void* q, void* out, void* stream)
{
    if (!valid_layer(p, layer) || !q || !out || !aligned16(q) || !aligned16(out)) return RLKV_EINVAL;
    int rc = check_slots(p, slots, n);
    if (rc) return rc;
    for (int i = 0; i < n; ++i)
        if (len_of(p, layer)[slots[i]] < 1) return RLKV_EEMPTY;
    DeviceGuard g(p->device);
    if (!g.ok) return RLKV_ECUDA;
    return paged_decode(p, layer, slots, n, q, out, static_cast<cudaStream_t>(stream), 0, false, 0, false, nullptr);
}

int rlkv_paged_step(rlkv_paged* p, const int* slots, int n, const void* k, const void* v, const void* q, void* out,
                    void* stream)
{
    if (!p || !k || !v || !q || !out || !aligned16(k) || !aligned16(v) || !aligned16(q) || !aligned16(out)) return RLKV_EINVAL;
    int rc = check_slots(p, slots, n);
    if (rc) return rc;
    // one append launch for all layers needs every listed sequence at the same length in every layer
    // (which is how a decode loop leaves them); room and pages are checked before anything changes
    int need = 0;
    for (int i = 0; i < n; ++i) {
        const int t = len_of(p, 0)[slots[i]];
        for (int l = 1; l < p->layers; ++l)
            if (len_of(p, l)[slots[i]] != t) return RLKV_EINVAL;
        if (t >= p->max_seq_len) return RLKV_EFULL;
        if (p->table[(size_t)slots[i] * p->table_stride + t / kTile] < 0) ++need;
    }
    if (need > (int)p->free_pages.size()) return RLKV_EFULL;
    if (p->layers > kMaxStepLayers) return RLKV_EINVAL;
    DeviceGuard g(p->device);
    if (!g.ok) return RLKV_ECUDA;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    PagedAppendArgs aa;
    fill_append_args(p, 0, k, v, aa);
    aa.prefill = 0;
    aa.n = n;
    aa.t0 = 0;
    aa.first_page = 0;
    aa.n_layers = p->layers;
    aa.layers = dev_at<LayerDesc>(p, p->off_layer_desc);
    for (int i = 0; i < n; ++i) {
        const int sl = slots[i], t = len_of(p, 0)[sl];
        int& entry = p->table[(size_t)sl * p->table_stride + t / kTile];
        if (entry < 0) {
            entry = p->free_pages.back();
            p->free_pages.pop_back();
        }
        aa.slot[i] = (unsigned short)sl;
        aa.t[i] = t;
        aa.page[i] = entry;
    }
    RLKV_CUDA(launch_paged_append(aa, s));
    p->launches++;
    for (int l = 0; l < p->layers; ++l)
        for (int i = 0; i < n; ++i) len_of(p, l)[slots[i]] += 1;
    // one decode launch over all layers (it may start beside the append launch and waits for it on the
    // device); where the step's partial records would not fit the scratch, or the caller asked for it,
    // one launch per layer, overlapped as in rlkv_step (step_launch_mode in rlkv_host.cuh)
    if (p->step_mode != 1 && p->step_in_one_launch && p->layers > 1) {  // (one layer: the per-layer launch is the whole step)
        rc = paged_decode(p, 0, slots, n, q, out, s, 0, true, 1, true, nullptr, true);
        if (rc != RLKV_ESCRATCH) return rc;
    }
    const size_t q_layer = (size_t)n * p->q_heads * p->head_dim;
    for (int l = 0; l < p->layers; ++l) {
        const StepLaunchMode m = step_launch_mode(l == 0, true);
        rc = paged_decode(p, l, slots, n, static_cast<const __nv_bfloat16*>(q) + l * q_layer,
                          static_cast<uint8_t*>(out) + l * q_layer * (p->out_bf16 ? 2 : 4), s, l & 1, m.overlap, m.dep_wait, true,
                          nullptr);
        if (rc) return rc;
    }
    return RLKV_OK;
}



int rlkv_paged_set_step_mode(rlkv_paged* p, int mode)
{
    if (!p || mode < 0 || mode > 2) return RLKV_EINVAL;
    if (mode == 2 && !p->step_in_one_launch) return RLKV_EINVAL;
    p->step_mode = mode;
    return RLKV_OK;
}

int rlkv_paged_set_output_bf16(rlkv_paged* p, int on)
{
    if (!p) return RLKV_EINVAL;
    p->out_bf16 = on ? 1 : 0;
    return RLKV_OK;
}

int rlkv_paged_length(const rlkv_paged* p, int layer, int slot, int* len_out)
{
    if (!valid_layer(p, layer) || !valid_slot(p, slot) || !len_out) return RLKV_EINVAL;
    *len_out = len_of(p, layer)[slot];
    return RLKV_OK;
}

int rlkv_paged_pages(const rlkv_paged* p, int* free_out, int* total_out)
{
    if (!p || !free_out || !total_out) return RLKV_EINVAL;
    *free_out = (int)p->free_pages.size();
    *total_out = p->n_pages;
    return RLKV_OK;
}

int rlkv_paged_step_bytes(const rlkv_paged* p, int layer, const int* slots, int n, uint64_t* kv_bytes_out)
{
    if (!valid_layer(p, layer) || !kv_bytes_out) return RLKV_EINVAL;
    int rc = check_slots(p, slots, n);
    if (rc) return rc;
    const int cap = p->sink + p->window;
    uint64_t rows = 0;
    for (int i = 0; i < n; ++i) {
        const int t = len_of(p, layer)[slots[i]];
        rows += (uint64_t)p->n_full[layer] * t + (uint64_t)p->n_comp[layer] * (t < cap ? t : cap);
    }
    *kv_bytes_out = rows * 2 * p->head_dim * (p->fp8 ? 1 : 2);  // a K row and a V row of codes or of bf16
    return RLKV_OK;
}

int rlkv_paged_debug_export_head(rlkv_paged* p, int layer, int slot, int kv_head, void* k_host, void* v_host,
                                 int* rows_out, int32_t* token_of_slot_host)
{
    if (!valid_layer(p, layer) || !valid_slot(p, slot) || kv_head < 0 || kv_head >= p->kv_heads || !k_host || !v_host ||
        !rows_out || !token_of_slot_host)
        return RLKV_EINVAL;
    DeviceGuard g(p->device);
    if (!g.ok) return RLKV_ECUDA;
    RLKV_CUDA(cudaDeviceSynchronize());
    const int n = len_of(p, layer)[slot], D = p->head_dim;
    const int s = p->slot_of_head[(size_t)layer * p->kv_heads + kv_head];
    const uint8_t* pool = p->dev_base + p->off_pool;
    const size_t row_bytes = (size_t)D * 2;
    if (s >= 0 && p->fp8) {  // a full head in 8-bit pages: its codes, one per 16-bit element of the output
        std::vector<uint8_t> page_bytes((size_t)2 * kTile * 128);
        uint16_t* kh = static_cast<uint16_t*>(k_host);
        uint16_t* vh = static_cast<uint16_t*>(v_host);
        for (int t0 = 0; t0 < n; t0 += kTile) {
            const int page = p->table[(size_t)slot * p->table_stride + t0 / kTile];
            if (page < 0) return RLKV_EKERNEL;
            const int cnt = n - t0 < kTile ? n - t0 : kTile;
            const uint8_t* src = p->dev_base + p->off_pool8 +
                                 (size_t)(p->page0_8[layer] + (long long)s * p->n_pages + page) * page_bytes.size();
            RLKV_CUDA(cudaMemcpy(page_bytes.data(), src, page_bytes.size(), cudaMemcpyDeviceToHost));
            for (int t = 0; t < cnt; ++t)
                for (int d = 0; d < D; ++d) {
                    kh[(size_t)(t0 + t) * D + d] = page_bytes[(size_t)t * 128 + d];
                    vh[(size_t)(t0 + t) * D + d] = page_bytes[(size_t)kTile * 128 + (size_t)d * kTile + t];  // transposed
                }
        }
        for (int t = 0; t < n; ++t) token_of_slot_host[t] = t;
        *rows_out = n;
    } else if (s >= 0) {  // a full head: its n tokens in token order, page by page
        for (int t0 = 0; t0 < n; t0 += kTile) {
            const int page = p->table[(size_t)slot * p->table_stride + t0 / kTile];
            if (page < 0) return RLKV_EKERNEL;
            const int cnt = n - t0 < kTile ? n - t0 : kTile;
            const long long krow = p->full_row0[layer] + ((long long)s * p->n_pages + page) * 2 * kTile;
            RLKV_CUDA(cudaMemcpy(static_cast<uint8_t*>(k_host) + t0 * row_bytes, pool + krow * row_bytes, cnt * row_bytes,
                                 cudaMemcpyDeviceToHost));
            RLKV_CUDA(cudaMemcpy(static_cast<uint8_t*>(v_host) + t0 * row_bytes, pool + (krow + kTile) * row_bytes,
                                 cnt * row_bytes, cudaMemcpyDeviceToHost));
        }
        for (int t = 0; t < n; ++t) token_of_slot_host[t] = t;
        *rows_out = n;
    } else if (p->fp8) {  // a compressed head in 8-bit storage: the codes of its physical ring
        const int cap = p->sink + p->window, ring_tiles = p->rows_comp / kTile;
        std::vector<uint8_t> page_bytes((size_t)2 * kTile * 128);
        uint16_t* kh = static_cast<uint16_t*>(k_host);
        uint16_t* vh = static_cast<uint16_t*>(v_host);
        for (int r0 = 0; r0 < cap; r0 += kTile) {
            const long long page = p->ring0_8[layer] + ((long long)slot * p->n_comp[layer] + (-s - 1)) * ring_tiles + r0 / kTile;
            RLKV_CUDA(cudaMemcpy(page_bytes.data(), p->dev_base + p->off_pool8 + (size_t)page * page_bytes.size(),
                                 page_bytes.size(), cudaMemcpyDeviceToHost));
            for (int r = 0; r < kTile && r0 + r < cap; ++r)
                for (int d = 0; d < D; ++d) {
                    kh[(size_t)(r0 + r) * D + d] = page_bytes[(size_t)r * 128 + d];
                    vh[(size_t)(r0 + r) * D + d] = page_bytes[(size_t)kTile * 128 + (size_t)d * kTile + r];
                }
        }
        for (int r = 0; r < cap; ++r) {
            int tok = -1;
            if (r < p->sink) {
                if (r < n) tok = r;
            } else if (n > p->sink) {
                const int newest = n - 1, back = ((newest - p->sink) - (r - p->sink)) % p->window;
                const int cand = newest - (back < 0 ? back + p->window : back);
                if (cand >= p->sink) tok = cand;
            }
            token_of_slot_host[r] = tok;
        }
        *rows_out = cap;
    } else {       // a compressed head: the physical ring
        const int cap = p->sink + p->window;
        const long long krow = p->comp_row0[layer] + ((long long)slot * p->n_comp[layer] + (-s - 1)) * 2 * p->rows_comp;
        RLKV_CUDA(cudaMemcpy(k_host, pool + krow * row_bytes, cap * row_bytes, cudaMemcpyDeviceToHost));
        RLKV_CUDA(cudaMemcpy(v_host, pool + (krow + p->rows_comp) * row_bytes, cap * row_bytes, cudaMemcpyDeviceToHost));
        for (int r = 0; r < cap; ++r) {
            int tok = -1;
            if (r < p->sink) {
                if (r < n) tok = r;
            } else if (n > p->sink) {
                // the newest token t >= sink with sink + (t - sink) % window == r
                const int newest = n - 1, back = ((newest - p->sink) - (r - p->sink)) % p->window;
                const int cand = newest - (back < 0 ? back + p->window : back);
                if (cand >= p->sink) tok = cand;
            }
            token_of_slot_host[r] = tok;
        }
        *rows_out = cap;
    }
    return RLKV_OK;
}

int rlkv_debug_paged_schedule(const int* lens, int n, int n_full, int n_comp, int cap, int ctas, int item_tiles,
                              int* n_items_out, int* delivered_out, int* expected_out, int* complete_out)
{
    if (!lens || n < 1 || n > kMaxPagedBatch || n_full < 0 || n_comp < 0 || n_full + n_comp < 1 || cap < 1 || ctas < 1 ||
        item_tiles < 1 || !n_items_out || !delivered_out || !expected_out || !complete_out)
        return RLKV_EINVAL;
    int longest = 0;
    for (int i = 0; i < n; ++i) {
        if (lens[i] < 1) return RLKV_EINVAL;
        if (lens[i] > longest) longest = lens[i];
    }
    const int tf = (longest + kTile - 1) / kTile, tc = ((longest < cap ? longest : cap) + kTile - 1) / kTile;
    const Schedule sc = make_schedule(n * n_full, tf, n * n_comp, tc, ctas, item_tiles);
    const int units = n * (n_full + n_comp);
    auto unit_tiles = [&](int uid) {  // tiles of the unit that exist
        int len = uid < sc.U ? lens[uid / n_full] : lens[(uid - sc.U) / n_comp];
        if (uid >= sc.U && len > cap) len = cap;
        return (len + kTile - 1) / kTile;
    };
    std::vector<int> last_slot(units, -1);
    for (int u = 0; u < units; ++u) delivered_out[u] = complete_out[u] = 0;
    // what the kernel does: walk every work item segment by segment
    for (int k = 0; k < sc.n_items; ++k) {
        const int x1 = item_start(sc, k + 1);
        for (int x = item_start(sc, k); x < x1;) {
            const TilePos pos = tile_pos(sc, x);
            const int seg_tiles = x1 - x < pos.run ? x1 - x : pos.run;
            const int exist = unit_tiles(pos.uid) - pos.tile;
            if (exist > 0) {
                if (pos.tile == 0 && seg_tiles >= unit_tiles(pos.uid)) {
                    complete_out[pos.uid]++;
                } else {
                    const int slot = partial_slot(sc, pos.band, k, pos.uid);
                    if (slot < 0 || slot >= sc.n_slots || slot <= last_slot[pos.uid]) return RLKV_EKERNEL;
                    last_slot[pos.uid] = slot;
                    delivered_out[pos.uid]++;
                }
            }
            x += seg_tiles;
        }
    }
    // what the tickets expect: the records of every band, clipped to the tiles that exist
    for (int u = 0; u < units; ++u) {
        int total = 0;
        for (int r = 0; r <= sc.R; ++r) {
            int slot = 0, count = 0;
            unit_partials(sc, u, r, slot, count, unit_tiles(u));
            total += count;
        }
        expected_out[u] = total;
    }
    *n_items_out = sc.n_items;
    return RLKV_OK;
}

int rlkv_paged_kernel_status(rlkv_paged* p, int* status_out)
{
    if (!p || !status_out) return RLKV_EINVAL;
    DeviceGuard g(p->device);
    if (!g.ok) return RLKV_ECUDA;
    RLKV_CUDA(cudaDeviceSynchronize());
    RLKV_CUDA(cudaMemcpy(status_out, p->dev_base + p->off_status, sizeof(int), cudaMemcpyDeviceToHost));
    return RLKV_OK;
}

}  // extern "C"
