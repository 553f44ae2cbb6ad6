// Fused append / bulk append: writes the new K and V rows of every (batch row, KV head) of one
// layer into the pool of the head's class and wraps the ring of compressed heads.
//
// Compressed-head slot rule: token t lives in row t if t < sink, else in row
// sink + ((t - sink) mod window) -- a constant-size circular buffer of sink + window rows holding
// the first `sink` tokens and the most recent `window` tokens (paper, Section 4.3 and Appendix B).
// In a bulk append only the tokens that survive the whole batch of appends are written, so no two
// threads ever target the same row and the result equals n successive single appends bit for bit.
#include <cuda_fp8.h>

#include "rlkv_internal.cuh"

namespace rlkv {
namespace {

__global__ void __launch_bounds__(256) append_kernel(const AppendArgs a)
{
    if (a.overlap) {  // launched so that it may start before the kernel that writes k and v has completed
        grid_dep_launch();  // the next kernel may start as well: it waits for this one before it reads the new rows
        grid_dep_wait();
    }
    const int chunks = a.head_dim / 8;  // 16-byte pieces per row
    const long long per_token = (long long)a.batch * a.kv_heads * chunks;
    const long long total = per_token * a.n_tokens * 2;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total;
         i += (long long)gridDim.x * blockDim.x) {
        long long r = i;
        const int c = (int)(r % chunks);
        r /= chunks;
        const int h = (int)(r % a.kv_heads);
        r /= a.kv_heads;
        const int b = (int)(r % a.batch);
        r /= a.batch;
        const int tok = (int)(r % a.n_tokens);
        const int kv = (int)(r / a.n_tokens);  // 0 = K, 1 = V

        const int t = a.t0 + tok;
        const int slot = a.slot_of_head[h];
        long long row;
        if (slot >= 0) {
            row = a.full_row0 + ((long long)(b * a.n_full + slot) * 2 + kv) * a.rows_full + t;
        } else {
            const int n_final = a.t0 + a.n_tokens;
            if (!(t < a.sink || t >= n_final - a.window)) continue;  // evicted before the batch ends
            const int phys = t < a.sink ? t : a.sink + (t - a.sink) % a.window;
            row = a.comp_row0 + ((long long)(b * a.n_comp + (-slot - 1)) * 2 + kv) * a.rows_comp + phys;
        }
        const __nv_bfloat16* src = (kv ? a.v : a.k) +
                                   (((long long)tok * a.batch + b) * a.kv_heads + h) * a.head_dim;
        const uint4 bits = __ldg(reinterpret_cast<const uint4*>(src) + c);
        reinterpret_cast<uint4*>(a.pool + row * a.head_dim)[c] = bits;
    }
}

// One token for every layer: the same row arithmetic, one more index.
__global__ void __launch_bounds__(256) append_all_kernel(const __grid_constant__ AppendAllArgs a)
{
    const int chunks = a.head_dim / 8;
    const long long per_layer = (long long)a.batch * a.kv_heads * chunks * 2;
    const long long total = per_layer * a.n_layers;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total;
         i += (long long)gridDim.x * blockDim.x) {
        long long r = i;
        const int c = (int)(r % chunks);
        r /= chunks;
        const int h = (int)(r % a.kv_heads);
        r /= a.kv_heads;
        const int b = (int)(r % a.batch);
        r /= a.batch;
        const int kv = (int)(r % 2);  // 0 = K, 1 = V
        const int l = (int)(r / 2);
        const LayerDesc d = a.layers[l];
        const int t = a.t0[l];
        const int slot = a.slot_of_head[l * a.kv_heads + h];
        long long row;
        if (slot >= 0) {
            row = d.full_row0 + ((long long)(b * d.n_full + slot) * 2 + kv) * a.rows_full + t;
        } else {
            const int phys = t < a.sink ? t : a.sink + (t - a.sink) % a.window;
            row = d.comp_row0 + ((long long)(b * d.n_comp + (-slot - 1)) * 2 + kv) * a.rows_comp + phys;
        }
        const __nv_bfloat16* src = (kv ? a.v : a.k) + (((long long)l * a.batch + b) * a.kv_heads + h) * a.head_dim;
        const uint4 bits = __ldg(reinterpret_cast<const uint4*>(src) + c);
        reinterpret_cast<uint4*>(a.pool + row * a.head_dim)[c] = bits;
    }
}

// Paged cache.  A full head's token t goes to row t % 64 of the sequence's page t / 64; a compressed
// head's to its ring slot (request slot instead of batch row).  The thread that writes the first piece
// of the row of the layer's first full head also records the page in the device page table (every
// token of a page and every layer write the same value there).
__global__ void __launch_bounds__(256) paged_append_kernel(const __grid_constant__ PagedAppendArgs a)
{
    const int chunks = a.head_dim / 8;
    const long long per_layer = (long long)a.n * a.kv_heads * chunks * 2;
    const long long total = per_layer * a.n_layers;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total;
         i += (long long)gridDim.x * blockDim.x) {
        const int l = (int)(i / per_layer);
        long long r = i - l * per_layer;
        const int c = (int)(r % chunks);
        r /= chunks;
        const int h = (int)(r % a.kv_heads);
        r /= a.kv_heads;
        const int e = (int)(r % a.n);   // entry of k, v
        const int kv = (int)(r / a.n);  // 0 = K, 1 = V
        const int seq = a.prefill ? a.slot[0] : a.slot[e];
        const int t = a.prefill ? a.t0 + e : a.t[e];
        const int page = a.page[a.prefill ? t / kTile - a.first_page : e];
        const int slot = a.slot_of_head[l * a.kv_heads + h];
        long long full_row0 = a.full_row0, comp_row0 = a.comp_row0;
        int n_comp = a.n_comp;
        if (a.n_layers > 1) {
            full_row0 = a.layers[l].full_row0;
            comp_row0 = a.layers[l].comp_row0;
            n_comp = a.layers[l].n_comp;
        }
        long long row;
        if (a.pool8) {
            // 8-bit pages: code = E4M3(x * (1 / scale)), round to nearest even, saturating.  A page is
            // the K codes [64 rows][128] followed by the V codes transposed [128][64 rows]; a full head's
            // token t is row t % 64 of the sequence's page t / 64, a compressed head's ring row r is row
            // r % 64 of page r / 64 of its ring.
            long long page_index;
            int prow;
            if (slot >= 0) {
                const long long page0 = a.n_layers > 1 ? a.layers[l].page0_8 : a.page0_8;
                page_index = page0 + (long long)slot * a.n_pages + page;
                prow = t % kTile;
            } else {
                if (a.prefill) {
                    const int n_final = a.t0 + a.n;
                    if (!(t < a.sink || t >= n_final - a.window)) continue;  // evicted before the batch ends
                }
                const int phys = t < a.sink ? t : a.sink + (t - a.sink) % a.window;
                const long long ring0 = a.n_layers > 1 ? a.layers[l].ring0_8 : a.ring0_8;
                page_index = ring0 + ((long long)seq * n_comp + (-slot - 1)) * a.ring_tiles + phys / kTile;
                prow = phys % kTile;
            }
            unsigned char* pg = a.pool8 + page_index * (2 * kTile * 128);
            const float inv = (kv ? a.v_inv : a.k_inv)[l * a.kv_heads + h];
            const __nv_bfloat16* src = (kv ? a.v : a.k) + ((long long)l * a.n + e) * a.entry_stride + (long long)h * a.head_dim + c * 8;
            const uint4 bits = __ldg(reinterpret_cast<const uint4*>(src));
            const __nv_bfloat16* x = reinterpret_cast<const __nv_bfloat16*>(&bits);
            alignas(8) unsigned char code[8];
#pragma unroll
            for (int j = 0; j < 8; ++j)
                code[j] = (unsigned char)__nv_cvt_float_to_fp8(__bfloat162float(x[j]) * inv, __NV_SATFINITE, __NV_E4M3);
            if (kv == 0) {
                *reinterpret_cast<uint2*>(pg + prow * 128 + c * 8) = *reinterpret_cast<const uint2*>(code);
            } else {
#pragma unroll
                for (int j = 0; j < 8; ++j) pg[kTile * 128 + (c * 8 + j) * kTile + prow] = code[j];
            }
            if (slot == 0 && c == 0 && kv == 0) a.page_table[(size_t)seq * a.table_stride + t / kTile] = page;
            continue;
        }
        if (slot >= 0) {
            row = full_row0 + (((long long)slot * a.n_pages + page) * 2 + kv) * kTile + t % kTile;
            if (slot == 0 && c == 0 && kv == 0) a.page_table[(size_t)seq * a.table_stride + t / kTile] = page;
        } else {
            if (a.prefill) {
                const int n_final = a.t0 + a.n;
                if (!(t < a.sink || t >= n_final - a.window)) continue;  // evicted before the batch ends
            }
            const int phys = t < a.sink ? t : a.sink + (t - a.sink) % a.window;
            row = comp_row0 + (((long long)seq * n_comp + (-slot - 1)) * 2 + kv) * a.rows_comp + phys;
        }
        const __nv_bfloat16* src = (kv ? a.v : a.k) + ((long long)l * a.n + e) * a.entry_stride + (long long)h * a.head_dim;
        const uint4 bits = __ldg(reinterpret_cast<const uint4*>(src) + c);
        reinterpret_cast<uint4*>(a.pool + row * a.head_dim)[c] = bits;
    }
}

}  // namespace

cudaError_t launch_paged_append(const PagedAppendArgs& a, cudaStream_t stream)
{
    const long long total = (long long)a.n_layers * a.n * a.kv_heads * (a.head_dim / 8) * 2;
    long long blocks = (total + 255) / 256;
    if (blocks > 148 * 16) blocks = 148 * 16;
    if (blocks < 1) blocks = 1;
    paged_append_kernel<<<(unsigned)blocks, 256, 0, stream>>>(a);
    return cudaGetLastError();
}

cudaError_t launch_append(const AppendArgs& a, cudaStream_t stream)
{
    const long long total = (long long)a.batch * a.kv_heads * (a.head_dim / 8) * a.n_tokens * 2;
    long long blocks = (total + 255) / 256;
    if (blocks > 148 * 16) blocks = 148 * 16;
    if (blocks < 1) blocks = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)blocks);
    cfg.blockDim = dim3(256);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = a.overlap ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, append_kernel, a);
}

cudaError_t launch_append_all(const AppendAllArgs& a, cudaStream_t stream)
{
    const long long total = (long long)a.n_layers * a.batch * a.kv_heads * (a.head_dim / 8) * 2;
    long long blocks = (total + 255) / 256;
    if (blocks > 148 * 8) blocks = 148 * 8;
    if (blocks < 1) blocks = 1;
    append_all_kernel<<<(unsigned)blocks, 256, 0, stream>>>(a);
    return cudaGetLastError();
}

}  // namespace rlkv
