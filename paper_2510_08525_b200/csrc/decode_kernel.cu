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
// with TMA (cp.async.bulk.tensor, 128-byte swizzle, mbarrier pipeline); four consumer warps each
// take 16 tokens of every tile: S = Q.K^T and O^T += V^T.P^T run on mma.sync m16n8k16 (bf16 in, fp32
// accumulate) with the G query heads of the group as the M (resp. N) dimension, online softmax in
// fp32 with warp shuffles.  The path is HBM-bound: the tensor-core work is ~G flop per byte.
// When a CTA's range ends inside a unit it writes an (m, l, O) partial; the last CTA to finish a
// unit (atomic ticket, no spinning) merges the partials with the log-sum-exp rule and writes out.
#include "rlkv_internal.cuh"

namespace rlkv {
namespace {

constexpr int kThreads = kConsumerThreads + 32;  // 4 consumer warps + 1 producer warp
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
__device__ __forceinline__ void consumer_sync()
{
    asm volatile("bar.sync 1, %0;" ::"n"(kConsumerThreads) : "memory");
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
template <int D>
struct Smem {
    static constexpr int kTileBytes = kTile * D * 2;       // one K (or V) tile
    static constexpr int kStageBytes = 2 * kTileBytes;     // K tile then V tile
    static constexpr int kMergeStride = D + kMergePad;     // floats per head row
    static constexpr int kMergeFloats = kConsumerWarps * kMaxGroup * kMergeStride;
    static constexpr int kStatFloats = 2 * kConsumerWarps * kMaxGroup;
    __host__ __device__ static constexpr size_t bytes(int stages)
    {
        return 1024 /*alignment slack*/ + (size_t)stages * kStageBytes + kMergeFloats * 4 +
               kStatFloats * 4 + 2 * 8 * 8 /*barriers*/ + 16 /*flags*/;
    }
};

// ---------------------------------------------------------------------------------------------
// End of a segment (the part of one unit a CTA processed).  Input: each consumer warp has put its
// running max / sum / un-normalised output into the merge area.  The 128 consumer threads merge the
// four warps; a complete unit is normalised and written out, otherwise the partial goes to the
// scratch buffer and the last CTA to arrive for that unit merges all partials of the unit.
template <int D>
__device__ void finalize_segment(const DecodeArgs& a, const UnitInfo& u, bool complete,
                                 const float* merge, const float* stat_m, const float* stat_l,
                                 int* s_flag, int ctid, int T, int P)
{
    constexpr int MS = Smem<D>::kMergeStride;
    constexpr int PF = partial_floats(D);
    const int G = a.group;
    consumer_sync();  // merge area written by all warps

    const int cta = blockIdx.x;
    const int my_slot = (cta_start(cta, T, P) >= u.first_tile) ? 0 : 1;
    float* my_part = a.partials + ((size_t)cta * 2 + my_slot) * PF;
    float* out_rows = a.out + ((size_t)u.b * a.q_heads + (size_t)u.head * G) * D;

    for (int idx = ctid; idx < G * D; idx += kConsumerThreads) {
        const int g = idx / D, d = idx - g * D;
        float M = kNegBig, L = 0.f, O = 0.f;
#pragma unroll
        for (int w = 0; w < kConsumerWarps; ++w) {
            const float mw = stat_m[w * kMaxGroup + g];
            const float lw = stat_l[w * kMaxGroup + g];
            const float ow = merge[(w * kMaxGroup + g) * MS + d];
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
        consumer_sync();
        if (ctid == 0) {
            const int old = atomicAdd(&a.tickets[u.unit], 1);
            *s_flag = (old == last_c - first_c);
        }
        consumer_sync();
        if (*s_flag) {
            __threadfence();
            for (int idx = ctid; idx < G * D; idx += kConsumerThreads) {
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
    consumer_sync();  // merge area and s_flag may be reused
}

// ---------------------------------------------------------------------------------------------
// The kernel.
template <int D>
__global__ void __launch_bounds__(kThreads, 1)
decode_kernel(const DecodeArgs a, const __grid_constant__ CUtensorMap tmap, const int stages)
{
    using S = Smem<D>;
    constexpr int KS = D / 16;  // k-steps of Q.K^T; also 16-row slabs of O^T
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                               ~static_cast<uintptr_t>(1023));
    uint8_t* stage_base = smem;
    float* merge = reinterpret_cast<float*>(smem + (size_t)stages * S::kStageBytes);
    float* stat_m = merge + S::kMergeFloats;
    float* stat_l = stat_m + kConsumerWarps * kMaxGroup;
    uint64_t* full_bar = reinterpret_cast<uint64_t*>(stat_l + kConsumerWarps * kMaxGroup);
    uint64_t* empty_bar = full_bar + 8;
    int* s_flag = reinterpret_cast<int*>(empty_bar + 8);
    volatile int* s_abort = s_flag + 1;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int T = a.total_tiles, P = gridDim.x;
    const int start = (int)cta_start(blockIdx.x, T, P);
    const int end = (int)cta_start(blockIdx.x + 1, T, P);

    if (tid == 0) {
        for (int s = 0; s < stages; ++s) {
            mbar_init(smem_u32(full_bar + s), 1);
            mbar_init(smem_u32(empty_bar + s), kConsumerWarps);
        }
        *s_flag = 0;
        *s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    if (warp == kConsumerWarps) {
        // ------------------------------------------------------------------ producer warp
        if (lane == 0) {
            asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap) : "memory");
            int it = 0;
            for (int x = start; x < end; ++x, ++it) {
                const UnitInfo u = locate(a, x);
                const int s = it % stages;
                const uint32_t par = (uint32_t)(it / stages) & 1u;
                wait_bounded(smem_u32(empty_bar + s), par ^ 1u, s_abort, a.status,
                             kStatusEmptyWaitTimeout);
                const uint32_t fb = smem_u32(full_bar + s);
                mbar_expect_tx(fb, S::kStageBytes);
                const uint32_t dst = smem_u32(stage_base + (size_t)s * S::kStageBytes);
                const int krow = (int)(u.krow + (long long)u.tile * kTile);
                const int vrow = krow + u.rows;
#pragma unroll
                for (int half = 0; half < D / 64; ++half) {
                    tma_load_2d(dst + half * (kTile * 128), &tmap, half * 64, krow, fb);
                    tma_load_2d(dst + S::kTileBytes + half * (kTile * 128), &tmap, half * 64, vrow,
                                fb);
                }
            }
        }
    } else {
        // ------------------------------------------------------------------ consumer warps
        const int quad = lane >> 2, tq = lane & 3;  // row inside an 8-row fragment, column pair
        const int ldm_j = lane >> 3, ldm_r = lane & 7;
        const int ldm_tok = warp * 16 + (ldm_j >> 1) * 8 + ldm_r;  // token row this lane addresses
        const int ldm_chunk = ldm_j & 1;                           // +1 16-byte chunk for odd matrices
        int it = 0;
        for (int x = start; x < end;) {
            const UnitInfo u = locate(a, x);
            const int seg_tiles = min(end - x, u.tiles - u.tile);

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

            for (int i = 0; i < seg_tiles; ++i, ++it) {
                const int s = it % stages;
                const uint32_t par = (uint32_t)(it / stages) & 1u;
                wait_bounded(smem_u32(full_bar + s), par, s_abort, a.status, kStatusFullWaitTimeout);
                const int valid = min(kTile, u.len - (u.tile + i) * kTile);
                if (warp * 16 < valid) {
                    const uint32_t sK = smem_u32(stage_base + (size_t)s * S::kStageBytes);
                    const uint32_t sV = sK + S::kTileBytes;
                    const uint32_t row_off = ldm_tok * 128;
                    // ---- S = Q.K^T for this warp's 16 tokens (two 8-token column blocks)
                    float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
                    float s2[4] = {0.f, 0.f, 0.f, 0.f}, s3[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                    for (int ks = 0; ks < KS; ++ks) {
                        const int chunk = ks * 2 + ldm_chunk;  // 16-byte chunk along d
                        const uint32_t addr = sK + (chunk >> 3) * (kTile * 128) + row_off +
                                              (((chunk & 7) ^ (ldm_tok & 7)) << 4);
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
                    // this lane: head `quad`, tokens warp*16 + {2tq, 2tq+1, 8+2tq, 9+2tq}
                    float sc[4];
                    sc[0] = (s0[0] + s2[0]) * a.scale_log2;
                    sc[1] = (s0[1] + s2[1]) * a.scale_log2;
                    sc[2] = (s1[0] + s3[0]) * a.scale_log2;
                    sc[3] = (s1[1] + s3[1]) * a.scale_log2;
                    const int tok0 = warp * 16 + 2 * tq;
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
                        const uint32_t addr = sV + (chunk >> 3) * (kTile * 128) + row_off +
                                              (((chunk & 7) ^ (ldm_tok & 7)) << 4);
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
                if (lane == 0) mbar_arrive(smem_u32(empty_bar + s));
            }

            // ---- hand the warp's state to the cross-warp merge
            l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
            l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
            if (tq == 0) {
                stat_m[warp * kMaxGroup + quad] = m_run;
                stat_l[warp * kMaxGroup + quad] = l_run;
            }
            {
                float* mw = merge + (size_t)warp * kMaxGroup * S::kMergeStride;
#pragma unroll
                for (int mt = 0; mt < KS; ++mt) {
                    const int d0 = mt * 16 + quad;
                    mw[(2 * tq) * S::kMergeStride + d0] = acc[mt][0];
                    mw[(2 * tq + 1) * S::kMergeStride + d0] = acc[mt][1];
                    mw[(2 * tq) * S::kMergeStride + d0 + 8] = acc[mt][2];
                    mw[(2 * tq + 1) * S::kMergeStride + d0 + 8] = acc[mt][3];
                }
            }
            finalize_segment<D>(a, u, u.tile == 0 && seg_tiles == u.tiles, merge, stat_m, stat_l,
                                s_flag, tid, T, P);
            x += seg_tiles;
        }
    }
    __syncthreads();
    if (warp == kConsumerWarps && lane == 0 && *s_abort) {
        // a wait ran out somewhere in this CTA: make sure none of its copies is still in flight
        // when the CTA retires
        const int issued = end - start;
        for (int j = issued > stages ? issued - stages : 0; j < issued; ++j)
            wait_bounded(smem_u32(full_bar + j % stages), (uint32_t)(j / stages) & 1u, s_abort, a.status,
                         kStatusDrainTimeout, false);
    }
}

// ---------------------------------------------------------------------------------------------
// Plain variant without TMA or tensor cores: direct global loads, CUDA-core FMAs, one token at a
// time per warp.  Same tile space, same partial/ticket protocol.  Kept as the debugging
// cross-check of the pipelined kernel (RLKV_DECODE_PLAIN=1 at cache creation); never the default.
template <int D>
__global__ void __launch_bounds__(kConsumerThreads, 2)
decode_kernel_plain(const DecodeArgs a)
{
    using S = Smem<D>;
    constexpr int DPL = D / 32;  // head_dim elements per lane
    __shared__ float merge[S::kMergeFloats];
    __shared__ float stat_m[kConsumerWarps * kMaxGroup];
    __shared__ float stat_l[kConsumerWarps * kMaxGroup];
    __shared__ int s_flag;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int T = a.total_tiles, P = gridDim.x;
    const int start = (int)cta_start(blockIdx.x, T, P);
    const int end = (int)cta_start(blockIdx.x + 1, T, P);
    const int G = a.group;

    for (int x = start; x < end;) {
        const UnitInfo u = locate(a, x);
        const int seg_tiles = min(end - x, u.tiles - u.tile);
        float qv[kMaxGroup][DPL], acc[kMaxGroup][DPL], m_run[kMaxGroup], l_run[kMaxGroup];
#pragma unroll
        for (int g = 0; g < kMaxGroup; ++g) {
            m_run[g] = kNegBig;
            l_run[g] = 0.f;
#pragma unroll
            for (int j = 0; j < DPL; ++j) {
                acc[g][j] = 0.f;
                qv[g][j] = g < G ? __bfloat162float(a.q[((size_t)u.b * a.q_heads + (size_t)u.head * G + g) * D +
                                                        lane * DPL + j])
                                 : 0.f;
            }
        }
        for (int i = 0; i < seg_tiles; ++i) {
            const int tile = u.tile + i;
            const int valid = min(kTile, u.len - tile * kTile);
            for (int r = warp * 16; r < min(warp * 16 + 16, valid); ++r) {
                const long long row = u.krow + (long long)tile * kTile + r;
                const __nv_bfloat16* kp = a.pool + row * D + lane * DPL;
                const __nv_bfloat16* vp = kp + (long long)u.rows * D;
                float kf[DPL], vf[DPL];
#pragma unroll
                for (int j = 0; j < DPL; ++j) {
                    kf[j] = __bfloat162float(kp[j]);
                    vf[j] = __bfloat162float(vp[j]);
                }
#pragma unroll
                for (int g = 0; g < kMaxGroup; ++g) {
                    if (g >= G) break;
                    float dot = 0.f;
#pragma unroll
                    for (int j = 0; j < DPL; ++j) dot += qv[g][j] * kf[j];
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
                    const float sc = dot * a.scale_log2;
                    const float m_new = fmaxf(m_run[g], sc);
                    const float corr = exp2f(m_run[g] - m_new), p = exp2f(sc - m_new);
                    l_run[g] = l_run[g] * corr + p;
                    m_run[g] = m_new;
#pragma unroll
                    for (int j = 0; j < DPL; ++j) acc[g][j] = acc[g][j] * corr + p * vf[j];
                }
            }
        }
#pragma unroll
        for (int g = 0; g < kMaxGroup; ++g) {
            if (lane == 0) {
                stat_m[warp * kMaxGroup + g] = m_run[g];
                stat_l[warp * kMaxGroup + g] = l_run[g];
            }
#pragma unroll
            for (int j = 0; j < DPL; ++j)
                merge[(warp * kMaxGroup + g) * S::kMergeStride + lane * DPL + j] = acc[g][j];
        }
        finalize_segment<D>(a, u, u.tile == 0 && seg_tiles == u.tiles, merge, stat_m, stat_l, &s_flag,
                            tid, T, P);
        x += seg_tiles;
    }
}

}  // namespace

size_t decode_smem_bytes(int head_dim, int stages)
{
    return head_dim == 128 ? Smem<128>::bytes(stages) : Smem<64>::bytes(stages);
}

cudaError_t prepare_decode_kernels(int head_dim, int stages)
{
    const int bytes = (int)decode_smem_bytes(head_dim, stages);
    if (head_dim == 128)
        return cudaFuncSetAttribute(decode_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    return cudaFuncSetAttribute(decode_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
}

cudaError_t launch_decode(const DecodeArgs& a, const CUtensorMap* tmap, int head_dim, int grid,
                          int stages, cudaStream_t stream)
{
    if (tmap == nullptr) {
        if (head_dim == 128)
            decode_kernel_plain<128><<<grid, kConsumerThreads, 0, stream>>>(a);
        else
            decode_kernel_plain<64><<<grid, kConsumerThreads, 0, stream>>>(a);
        return cudaGetLastError();
    }
    const size_t smem = decode_smem_bytes(head_dim, stages);
    if (head_dim == 128)
        decode_kernel<128><<<grid, kThreads, smem, stream>>>(a, *tmap, stages);
    else
        decode_kernel<64><<<grid, kThreads, smem, stream>>>(a, *tmap, stages);
    return cudaGetLastError();
}

}  // namespace rlkv
