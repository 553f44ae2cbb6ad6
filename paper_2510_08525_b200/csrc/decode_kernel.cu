// Split-KV decode attention over the heterogeneous heads of one layer, for sm_100a.
//
// What it computes (paper, Section 3.3 last paragraph): for every query head j of every batch row,
// softmax(q_j . K_h^T / sqrt(D)) . V_h over the rows KV head h = j / G retains -- all n tokens for a
// full head, the sink + ring rows for a compressed head.  One launch serves both head classes
// (the fused heterogeneous-head kernel Section 4.3 asks for).
//
// How: the K/V rows to read are cut into 64-token tiles and laid out as one flat tile space (full
// units first, compressed units after).  A persistent grid splits that space evenly: CTA c owns the
// contiguous range [c*T/P, (c+1)*T/P), so long full-head scans and short compressed-head scans
// balance to within one tile.  Inside a CTA one producer warp streams tiles HBM -> shared memory
// with TMA (cp.async.bulk.tensor, 128-byte swizzle, mbarrier pipeline); NG groups of four consumer
// warps take the tiles in turn, each warp 16 tokens of its group's tile: S = Q.K^T and
// O^T += V^T.P^T run on mma.sync m16n8k16 (bf16 in, fp32 accumulate) with the G query heads of the
// group as the M (resp. N) dimension, online softmax in fp32 with warp shuffles.  The path is
// HBM-bound (the tensor-core work is ~G flop per byte); several groups are there only to hide the
// dependent-issue latency of one tile's softmax chain behind another tile's.
// When a CTA's range ends inside a unit it writes an (m, l, O) partial; the last CTA to finish a
// unit (atomic ticket, no spinning) merges the partials with the log-sum-exp rule and writes out.
#include "rlkv_internal.cuh"

namespace rlkv {
namespace {

constexpr float kNegBig = -1.0e30f;              // finite "minus infinity" for running maxima

// ---------------------------------------------------------------------------------------------
// PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p)
{
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ uint64_t global_timer_ns()
{
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y,
                                            uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
        "l"(map), "r"(x), "r"(y), "r"(bar)
        : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int x, int y, int z,
                                            uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%2, %3, %4}], [%5];" ::"r"(dst),
        "l"(map), "r"(x), "r"(y), "r"(z), "r"(bar)
        : "memory");
}
// Byte offset inside a tile row of 16-byte chunk `chunk` of row `row` under the 128-byte swizzle.
template <int D>
__device__ __forceinline__ uint32_t swizzled_chunk(int row, int chunk)
{
    if (D == 128) return (uint32_t)(((chunk & 8) | ((chunk & 7) ^ ((2 * row + (chunk >> 3)) & 7))) << 4);
    return (uint32_t)((chunk ^ (row & 7)) << 4);
}
template <int NG>
__device__ __forceinline__ void consumer_sync()
{
    asm volatile("bar.sync 1, %0;" ::"n"(NG * kGroupWarps * 32) : "memory");
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2,
                                            uint32_t& r3)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1,
                                                  uint32_t& r2, uint32_t& r3)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                         uint32_t a3, uint32_t b0, uint32_t b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, "
        "{%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

// Wait on an mbarrier phase with a time limit (about one second).  When the limit runs out the
// kernel records `code` in the status word and raises the CTA-wide abort flag; every later wait
// then returns at once, so the CTA runs to its end (with meaningless results) instead of hanging.
__device__ __forceinline__ void wait_bounded(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                             int* status, int code, bool abortable = true)
{
    uint64_t t0 = 0;
    for (uint32_t i = 0;; ++i) {
        if (mbar_try_wait(bar, parity)) return;
        if (i < 128) continue;
        if (abortable && *abort_flag) return;
        __nanosleep(64);
        const uint64_t now = global_timer_ns();
        if (t0 == 0) {
            t0 = now;
        } else if (now - t0 > 1000000000ull) {
            atomicCAS(status, kStatusOk, code);
            *abort_flag = 1;
            return;
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Shared-memory carve-up (dynamic shared memory, base aligned to 1024 bytes for the swizzle).
template <int D, int NG>
struct Smem {
    static constexpr int kWarps = NG * kGroupWarps;         // consumer warps
    static constexpr int kTileBytes = kTile * D * 2;        // one K (or V) tile
    static constexpr int kStageBytes = 2 * kTileBytes;      // K tile then V tile
    static constexpr int kMergeStride = D + kMergePad;      // floats per head row
    static constexpr int kStatFloats = 2 * kWarps * kMaxGroup;
    __host__ __device__ static constexpr int merge_floats(int group) { return kWarps * group * kMergeStride; }
    __host__ __device__ static constexpr size_t bytes(int stages, int group)
    {
        return 1024 /*alignment slack*/ + (size_t)stages * kStageBytes + merge_floats(group) * 4 +
               kStatFloats * 4 + 2 * 8 * 8 /*barriers*/ + 16 /*flags*/;
    }
};

// ---------------------------------------------------------------------------------------------
// End of a segment (the part of one unit a CTA processed).  Input: each consumer warp has put its
// running max / sum / un-normalised output into the merge area.  The consumer threads merge the
// warps; a complete unit is normalised and written out, otherwise the partial goes to the scratch
// buffer and the last CTA to arrive for that unit merges all partials of the unit.
template <int D, int NG>
__device__ void finalize_segment(const DecodeArgs& a, const UnitInfo& u, bool complete,
                                 const float* merge, const float* stat_m, const float* stat_l,
                                 int* s_flag, int ctid)
{
    const int T = a.full_tiles, P = a.grid_full;  // the split space of the full units
    using S = Smem<D, NG>;
    constexpr int MS = S::kMergeStride;
    constexpr int PF = partial_floats(D);
    constexpr int NT = S::kWarps * 32;
    const int G = a.group;
    consumer_sync<NG>();  // merge area written by all warps

    const int cta = blockIdx.x;
    const int my_slot = (complete || cta_start(cta, T, P) >= u.first_tile) ? 0 : 1;
    float* my_part = a.partials + ((size_t)cta * 2 + my_slot) * PF;
    float* out_rows = a.out + ((size_t)u.b * a.q_heads + (size_t)u.head * G) * D;

    for (int idx = ctid; idx < G * D; idx += NT) {
        const int g = idx / D, d = idx - g * D;
        float M = kNegBig, L = 0.f, O = 0.f;
#pragma unroll
        for (int w = 0; w < S::kWarps; ++w) {
            const float mw = stat_m[w * kMaxGroup + g];
            const float lw = stat_l[w * kMaxGroup + g];
            const float ow = merge[(w * G + g) * MS + d];
            const float Mn = fmaxf(M, mw);
            const float ca = exp2f(M - Mn), cb = exp2f(mw - Mn);
            L = L * ca + lw * cb;
            O = O * ca + ow * cb;
            M = Mn;
        }
        if (complete) {
            out_rows[idx] = O / L;
        } else {
            my_part[2 * kMaxGroup + idx] = O;
            if (d == 0) {
                my_part[g] = M;
                my_part[kMaxGroup + g] = L;
            }
        }
    }
    if (!complete) {
        const int first_c = cta_of_tile(u.first_tile, T, P);
        const int last_c = cta_of_tile((long long)u.first_tile + u.tiles - 1, T, P);
        __threadfence();
        consumer_sync<NG>();
        if (ctid == 0) {
            const int old = atomicAdd(&a.tickets[u.unit], 1);
            *s_flag = (old == last_c - first_c);
        }
        consumer_sync<NG>();
        if (*s_flag) {
            __threadfence();
            for (int idx = ctid; idx < G * D; idx += NT) {
                const int g = idx / D;
                float M = kNegBig, L = 0.f, O = 0.f;
                for (int c = first_c; c <= last_c; ++c) {
                    const int slot = (cta_start(c, T, P) >= u.first_tile) ? 0 : 1;
                    const float* part = a.partials + ((size_t)c * 2 + slot) * PF;
                    const float mc = __ldcg(part + g);
                    const float lc = __ldcg(part + kMaxGroup + g);
                    const float oc = __ldcg(part + 2 * kMaxGroup + idx);
                    const float Mn = fmaxf(M, mc);
                    const float ca = exp2f(M - Mn), cb = exp2f(mc - Mn);
                    L = L * ca + lc * cb;
                    O = O * ca + oc * cb;
                    M = Mn;
                }
                out_rows[idx] = O / L;
            }
            if (ctid == 0) a.tickets[u.unit] = 0;  // ready for the next launch
        }
    }
    consumer_sync<NG>();  // merge area and s_flag may be reused
}

// ---------------------------------------------------------------------------------------------
// The kernel.  Warps 0 .. 4*NG-1 are consumers (group = warp / 4), the last warp is the producer.
template <int D, int NG>
__global__ void __launch_bounds__(NG * kGroupWarps * 32 + 32, 1)
decode_kernel(const DecodeArgs a, const __grid_constant__ CUtensorMap tmap, const int stages)
{
    using S = Smem<D, NG>;
    constexpr int KS = D / 16;  // k-steps of Q.K^T; also 16-row slabs of O^T
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                               ~static_cast<uintptr_t>(1023));
    uint8_t* stage_base = smem;
    float* merge = reinterpret_cast<float*>(smem + (size_t)stages * S::kStageBytes);
    float* stat_m = merge + S::merge_floats(a.group);
    float* stat_l = stat_m + S::kWarps * kMaxGroup;
    uint64_t* full_bar = reinterpret_cast<uint64_t*>(stat_l + S::kWarps * kMaxGroup);
    uint64_t* empty_bar = full_bar + 8;
    int* s_flag = reinterpret_cast<int*>(empty_bar + 8);
    volatile int* s_abort = s_flag + 1;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const CtaWork work = cta_work(a, blockIdx.x, gridDim.x);
    const bool stamp = (a.debug & 4) != 0;
    if (stamp && tid == 0) a.timeline[blockIdx.x * 4 + 0] = global_timer_ns();

    if (tid == 0) {
        for (int s = 0; s < stages; ++s) {
            mbar_init(smem_u32(full_bar + s), 1);
            mbar_init(smem_u32(empty_bar + s), kGroupWarps);
        }
        *s_flag = 0;
        *s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    if (warp == S::kWarps) {
        // ------------------------------------------------------------------ producer warp
        if (lane == 0) {
            asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap) : "memory");
            int s = 0;
            uint32_t par = 0;
            for (int v = 0; v < work.total; ++v) {
                const UnitInfo u = locate(a, work, v);
                wait_bounded(smem_u32(empty_bar + s), par ^ 1u, s_abort, a.status,
                             kStatusEmptyWaitTimeout);
                const uint32_t fb = smem_u32(full_bar + s);
                mbar_expect_tx(fb, S::kStageBytes);
                const uint32_t dst = smem_u32(stage_base + (size_t)s * S::kStageBytes);
                const int krow = (int)(u.krow + (long long)u.tile * kTile);
                const int vrow = krow + u.rows;
                if (D == 128) {  // one contiguous 16 KB box per tile: [64 rows][2 halves][64]
                    tma_load_3d(dst, &tmap, 0, 0, krow, fb);
                    tma_load_3d(dst + S::kTileBytes, &tmap, 0, 0, vrow, fb);
                } else {         // one contiguous 8 KB box per tile: [64 rows][64]
                    tma_load_2d(dst, &tmap, 0, krow, fb);
                    tma_load_2d(dst + S::kTileBytes, &tmap, 0, vrow, fb);
                }
                if (++s == stages) {
                    s = 0;
                    par ^= 1u;
                }
            }
        }
    } else {
        // ------------------------------------------------------------------ consumer warps
        const int grp = warp / kGroupWarps, wig = warp % kGroupWarps;  // tile group, 16-token slice
        const int quad = lane >> 2, tq = lane & 3;  // row inside an 8-row fragment, column pair
        const int ldm_j = lane >> 3, ldm_r = lane & 7;
        const int ldm_tok = wig * 16 + (ldm_j >> 1) * 8 + ldm_r;  // token row this lane addresses
        const int ldm_chunk = ldm_j & 1;                          // +1 16-byte chunk for odd matrices
        // Tile layout in shared memory (written by TMA with the 128-byte swizzle): row r of the tile
        // starts at r*2*D bytes; its 16-byte chunk c sits at chunk index c ^ (bits 7..9 of the
        // unswizzled offset), i.e. c ^ ((2r + c/8) & 7) for D = 128 and c ^ (r & 7) for D = 64.
        const uint32_t row_off = ldm_tok * (2 * D);
        int s = 0, turn = 0;  // pipeline stage and whose turn the next tile is
        uint32_t par = 0;
        for (int v = 0; v < work.total;) {
            const UnitInfo u = locate(a, work, v);
            const int seg_tiles = min(work.total - v, u.tiles - u.tile);

            // Q as the A operand (rows = query heads of the group, rows >= G are zero)
            uint32_t qa[KS][2];
            {
                const __nv_bfloat16* qrow =
                    a.q + ((size_t)u.b * a.q_heads + (size_t)u.head * a.group + quad) * D + 2 * tq;
#pragma unroll
                for (int ks = 0; ks < KS; ++ks) {
                    qa[ks][0] = quad < a.group ? *reinterpret_cast<const uint32_t*>(qrow + ks * 16) : 0u;
                    qa[ks][1] = quad < a.group ? *reinterpret_cast<const uint32_t*>(qrow + ks * 16 + 8) : 0u;
                }
            }
            float m_run = kNegBig, l_run = 0.f;
            float acc[KS][4];
#pragma unroll
            for (int mt = 0; mt < KS; ++mt) acc[mt][0] = acc[mt][1] = acc[mt][2] = acc[mt][3] = 0.f;

            int valid_left = u.len - u.tile * kTile;  // valid rows from this tile to the unit's end
            for (int i = 0; i < seg_tiles; ++i, valid_left -= kTile) {
                const bool mine = (turn == grp);
                const int cur_s = s;
                const uint32_t cur_par = par;
                if (++turn == NG) turn = 0;
                if (++s == stages) {
                    s = 0;
                    par ^= 1u;
                }
                if (!mine) continue;
                wait_bounded(smem_u32(full_bar + cur_s), cur_par, s_abort, a.status, kStatusFullWaitTimeout);
                if (stamp && tid == 0 && v == 0 && i == 0) a.timeline[blockIdx.x * 4 + 1] = global_timer_ns();
                const int valid = min(kTile, valid_left);
                if (wig * 16 < valid) {
                    const uint32_t sK = smem_u32(stage_base + (size_t)cur_s * S::kStageBytes);
                    const uint32_t sV = sK + S::kTileBytes;
                    // ---- S = Q.K^T for this warp's 16 tokens (two 8-token column blocks)
                    float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
                    float s2[4] = {0.f, 0.f, 0.f, 0.f}, s3[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                    for (int ks = 0; ks < KS; ++ks) {
                        const int chunk = ks * 2 + ldm_chunk;  // 16-byte chunk along d
                        const uint32_t addr = sK + row_off + swizzled_chunk<D>(ldm_tok, chunk);
                        uint32_t b0, b1, b2, b3;
                        ldmatrix_x4(addr, b0, b1, b2, b3);
                        if (ks & 1) {
                            mma_bf16(s2, qa[ks][0], 0u, qa[ks][1], 0u, b0, b1);
                            mma_bf16(s3, qa[ks][0], 0u, qa[ks][1], 0u, b2, b3);
                        } else {
                            mma_bf16(s0, qa[ks][0], 0u, qa[ks][1], 0u, b0, b1);
                            mma_bf16(s1, qa[ks][0], 0u, qa[ks][1], 0u, b2, b3);
                        }
                    }
                    // this lane: head `quad`, tokens wig*16 + {2tq, 2tq+1, 8+2tq, 9+2tq}
                    float sc[4];
                    sc[0] = (s0[0] + s2[0]) * a.scale_log2;
                    sc[1] = (s0[1] + s2[1]) * a.scale_log2;
                    sc[2] = (s1[0] + s3[0]) * a.scale_log2;
                    sc[3] = (s1[1] + s3[1]) * a.scale_log2;
                    const int tok0 = wig * 16 + 2 * tq;
                    if (tok0 >= valid) sc[0] = -INFINITY;
                    if (tok0 + 1 >= valid) sc[1] = -INFINITY;
                    if (tok0 + 8 >= valid) sc[2] = -INFINITY;
                    if (tok0 + 9 >= valid) sc[3] = -INFINITY;
                    // ---- online softmax (log2 domain)
                    float mx = fmaxf(fmaxf(sc[0], sc[1]), fmaxf(sc[2], sc[3]));
                    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
                    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
                    const float m_new = fmaxf(m_run, mx);
                    const float corr = exp2f(m_run - m_new);
                    const float p0 = exp2f(sc[0] - m_new), p1 = exp2f(sc[1] - m_new);
                    const float p2 = exp2f(sc[2] - m_new), p3 = exp2f(sc[3] - m_new);
                    l_run = l_run * corr + ((p0 + p1) + (p2 + p3));
                    m_run = m_new;
                    // O^T columns of this lane are heads 2tq and 2tq+1: fetch their corrections
                    const float ca = __shfl_sync(0xffffffffu, corr, tq * 8);
                    const float cb = __shfl_sync(0xffffffffu, corr, tq * 8 + 4);
                    const uint32_t pb0 = pack_bf16(p0, p1), pb1 = pack_bf16(p2, p3);
                    // ---- O^T[d][head] += V^T[d][tok] . P^T[tok][head]
#pragma unroll
                    for (int mt = 0; mt < KS; ++mt) {
                        const int chunk = mt * 2 + ldm_chunk;
                        const uint32_t addr = sV + row_off + swizzled_chunk<D>(ldm_tok, chunk);
                        uint32_t v0, v1, v2, v3;
                        ldmatrix_x4_trans(addr, v0, v1, v2, v3);
                        acc[mt][0] *= ca;
                        acc[mt][1] *= cb;
                        acc[mt][2] *= ca;
                        acc[mt][3] *= cb;
                        mma_bf16(acc[mt], v0, v1, v2, v3, pb0, pb1);
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(empty_bar + cur_s));
            }

            // ---- hand the warp's state to the cross-warp merge
            l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
            l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
            if (tq == 0) {
                stat_m[warp * kMaxGroup + quad] = m_run;
                stat_l[warp * kMaxGroup + quad] = l_run;
            }
            {
                const int G = a.group;
                float* mw = merge + (size_t)warp * G * S::kMergeStride;
                const int h0 = 2 * tq, h1 = 2 * tq + 1;
#pragma unroll
                for (int mt = 0; mt < KS; ++mt) {
                    const int d0 = mt * 16 + quad;
                    if (h0 < G) {
                        mw[h0 * S::kMergeStride + d0] = acc[mt][0];
                        mw[h0 * S::kMergeStride + d0 + 8] = acc[mt][2];
                    }
                    if (h1 < G) {
                        mw[h1 * S::kMergeStride + d0] = acc[mt][1];
                        mw[h1 * S::kMergeStride + d0 + 8] = acc[mt][3];
                    }
                }
            }
            if (stamp && tid == 0 && v + seg_tiles == work.total) a.timeline[blockIdx.x * 4 + 2] = global_timer_ns();
            finalize_segment<D, NG>(a, u, u.tile == 0 && seg_tiles == u.tiles, merge, stat_m, stat_l,
                                    s_flag, tid);
            v += seg_tiles;
        }
    }
    __syncthreads();
    if (stamp && tid == 0) a.timeline[blockIdx.x * 4 + 3] = global_timer_ns();
    if (warp == S::kWarps && lane == 0 && *s_abort) {
        // a wait ran out somewhere in this CTA: make sure none of its copies is still in flight
        // when the CTA retires
        const int issued = work.total;
        for (int j = issued > stages ? issued - stages : 0; j < issued; ++j)
            wait_bounded(smem_u32(full_bar + j % stages), (uint32_t)(j / stages) & 1u, s_abort, a.status,
                         kStatusDrainTimeout, false);
    }
}

template <int D, int NG>
cudaError_t launch_one(const DecodeArgs& a, const CUtensorMap& tmap, int grid, int stages, cudaStream_t stream)
{
    const size_t smem = Smem<D, NG>::bytes(stages, a.group);
    decode_kernel<D, NG><<<grid, NG * kGroupWarps * 32 + 32, smem, stream>>>(a, tmap, stages);
    return cudaGetLastError();
}

template <int D, int NG>
cudaError_t prepare_one()
{
    return cudaFuncSetAttribute(decode_kernel<D, NG>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                kMaxDynamicSmem);
}

}  // namespace

size_t decode_smem_bytes(int head_dim, int stages, int group, int groups)
{
    if (head_dim == 128)
        return groups == 1 ? Smem<128, 1>::bytes(stages, group)
                           : groups == 2 ? Smem<128, 2>::bytes(stages, group) : Smem<128, 3>::bytes(stages, group);
    return groups == 1 ? Smem<64, 1>::bytes(stages, group)
                       : groups == 2 ? Smem<64, 2>::bytes(stages, group) : Smem<64, 3>::bytes(stages, group);
}

cudaError_t prepare_decode_kernels(int head_dim)
{
    cudaError_t e;
    if (head_dim == 128) {
        if ((e = prepare_one<128, 1>()) != cudaSuccess) return e;
        if ((e = prepare_one<128, 2>()) != cudaSuccess) return e;
        return prepare_one<128, 3>();
    }
    if ((e = prepare_one<64, 1>()) != cudaSuccess) return e;
    if ((e = prepare_one<64, 2>()) != cudaSuccess) return e;
    return prepare_one<64, 3>();
}

cudaError_t launch_decode(const DecodeArgs& a, const CUtensorMap* tmap, int head_dim, int grid,
                          int stages, int groups, cudaStream_t stream)
{
    if (head_dim == 128) {
        if (groups == 1) return launch_one<128, 1>(a, *tmap, grid, stages, stream);
        if (groups == 2) return launch_one<128, 2>(a, *tmap, grid, stages, stream);
        return launch_one<128, 3>(a, *tmap, grid, stages, stream);
    }
    if (groups == 1) return launch_one<64, 1>(a, *tmap, grid, stages, stream);
    if (groups == 2) return launch_one<64, 2>(a, *tmap, grid, stages, stream);
    return launch_one<64, 3>(a, *tmap, grid, stages, stream);
}

}  // namespace rlkv
