// Split-KV decode attention over the heterogeneous heads of one layer, for sm_100a.
//
// What it computes (paper, Section 3.3 last paragraph): for every query head j of every batch row,
// softmax(q_j . K_h^T / sqrt(D)) . V_h over the rows KV head h = j / G retains -- all n tokens for a
// full head, the sink + ring rows for a compressed head.  One launch serves both head classes
// (the fused heterogeneous-head kernel Section 4.3 asks for).
//
// How: the K/V rows to read are cut into 64-token tiles and laid out as one flat tile space, which
// is cut into contiguous work items whose size shrinks geometrically (rlkv_internal.cuh); a
// persistent grid takes item c for CTA c and claims further items from an atomic counter, so long
// full-head scans and short compressed-head scans balance even though some SMs sit on a slower path
// to memory than others.  Inside a CTA one producer warp streams tiles HBM -> shared memory with TMA
// (cp.async.bulk.tensor, 128-byte swizzle, mbarrier pipeline); NG groups of four consumer warps take
// the tiles in turn, each warp 16 tokens of its group's tile: S = Q.K^T and O^T += V^T.P^T run on
// mma.sync m16n8k16 (bf16 in, fp32 accumulate) with the G query heads of the group as the M (resp. N)
// dimension, online softmax in fp32 with warp shuffles.  The path is HBM-bound (the tensor-core work
// is ~G flop per byte).
// When an item begins or ends inside a unit the CTA writes an (m, l, O) partial; the last CTA to
// deliver a partial of a unit (atomic ticket, no spinning) merges them with the log-sum-exp rule.
// The merge of the consumer warps' own states at the end of every segment and the tickets run on
// separate epilogue warps, so the tile stream never waits for a round trip to global memory; the
// merges of split units run on all warps once the CTA's stream has ended.
// The decode launches of one step overlap on the device (programmatic dependent launch): see the
// kernel's first lines and launch_decode.
// The kernel is compiled in several modes: the lock-step cache (above), mixed attention with gating
// adapters (paper, Eq. 1: a second class of "local" units over the sink and window rows, both
// classes adding their weighted result), the paged cache (one length per sequence, full-head
// rows looked up in a page table; also with 8-bit pages), and the whole decode step in one launch
// (the units of every layer in one flat tile space); see the notes above decode_kernel.
#include <cuda_fp16.h>
#include <stddef.h>

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
// L2 policy for data that is read once: K/V tiles stream through the L2 without pushing out the
// split-KV partials, tickets and query rows that are about to be read again.
__device__ __forceinline__ uint64_t l2_evict_first_policy()
{
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar,
                                            uint64_t policy)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint"
        " [%0], [%1, {%2, %3}], [%4], %5;" ::"r"(dst),
        "l"(map), "r"(x), "r"(y), "r"(bar), "l"(policy)
        : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int x, int y, int z, uint32_t bar,
                                            uint64_t policy)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint"
        " [%0], [%1, {%2, %3, %4}], [%5], %6;" ::"r"(dst),
        "l"(map), "r"(x), "r"(y), "r"(z), "r"(bar), "l"(policy)
        : "memory");
}
// Untiled bulk copy global -> shared (both addresses 16-byte aligned, size a multiple of 16).
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}
// Byte offset inside a K or V tile of 16-byte chunk `chunk` (along d) of token row `row`.  A tile
// is stored as D/64 blocks of [64 rows][128 bytes], written by TMA with the 128-byte swizzle: inside a
// block, chunk c of row r sits at chunk position c ^ (r & 7), so the eight rows of an ldmatrix
// fragment fall into eight different bank groups.
template <int D>
__device__ __forceinline__ uint32_t tile_offset(int row, int chunk)
{
    return (uint32_t)((chunk >> 3) * (kTile * 128) + row * 128 + (((chunk & 7) ^ (row & 7)) << 4));
}
// Barrier over the epilogue warps (named barrier 2).
__device__ __forceinline__ void epilogue_sync()
{
    asm volatile("bar.sync 2, %0;" ::"n"(kEpilogueWarps * 32) : "memory");
}
// The same barrier, also ORing a flag: every epilogue thread learns whether any of them gave up on
// a wait, so that they all leave together and the named barrier is never left short.
__device__ __forceinline__ bool epilogue_or(bool flag)
{
    uint32_t any;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 q, %1, 0;\n\t"
        "bar.red.or.pred p, 2, %2, q;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(any)
        : "r"((uint32_t)flag), "n"(kEpilogueWarps * 32)
        : "memory");
    return any != 0;
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
__device__ __forceinline__ void mma_f16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                        uint32_t b0, uint32_t b1)
{
    asm(  // no side effects: the compiler may schedule it among the conversions around it
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, "
        "{%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// Four E4M3 codes (one 32-bit register, lowest byte first) as two f16x2 registers: codes 0, 1 and
// codes 2, 3.  Every E4M3 value is an f16 value, so the conversion is exact.
__device__ __forceinline__ void e4m3x4_to_f16x2x2(uint32_t codes, uint32_t& lo, uint32_t& hi)
{
    asm(
        "{\n\t.reg .b16 a, b;\n\t"
        "mov.b32 {a, b}, %2;\n\t"
        "cvt.rn.f16x2.e4m3x2 %0, a;\n\t"
        "cvt.rn.f16x2.e4m3x2 %1, b;\n\t}"
        : "=r"(lo), "=r"(hi)
        : "r"(codes));
}
// Transposes an 8x8 matrix of 16-bit elements held one row per quad of lanes (lane l: row l / 4,
// columns 2(l % 4) and 2(l % 4) + 1): afterwards the lane holds the same positions of the transpose.
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a)
{
    uint32_t d;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
    return d;
}
__device__ __forceinline__ uint32_t pack_f16(float lo, float hi)
{
    __half2 v = __floats2half2_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

// Wait on an mbarrier phase with a time limit (about one second).  Returns true when the phase
// completed.  When the limit runs out the kernel records `code` in the status word, raises the
// CTA-wide abort flag and returns false; every later abortable wait of the CTA then gives up at
// once, so the CTA winds down (with meaningless results) instead of hanging.
__device__ __forceinline__ bool wait_bounded(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                             int* status, int code, bool abortable = true)
{
    uint64_t t0 = 0;
    for (uint32_t i = 0;; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if (i < 128) continue;
        if (abortable && *abort_flag) return false;
        __nanosleep(64);
        const uint64_t now = global_timer_ns();
        if (t0 == 0) {
            t0 = now;
        } else if (now - t0 > 1000000000ull) {
            atomicCAS(status, kStatusOk, code);
            *abort_flag = 1;
            return false;
        }
    }
}

// wait_bounded that also adds the SM clock cycles spent waiting to *cycles when the trace is on (one
// thread's view; the cycle counter is cheap to read, unlike %globaltimer).
__device__ __forceinline__ bool wait_traced(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status,
                                            int code, bool on, unsigned long long* cycles)
{
    if (!on) return wait_bounded(bar, parity, abort_flag, status, code);
    const long long t = clock64();
    const bool ok = wait_bounded(bar, parity, abort_flag, status, code);
    *cycles += (unsigned long long)(clock64() - t);
    return ok;
}

// ---------------------------------------------------------------------------------------------
// What the consumer warps tell the epilogue warps about a finished segment (the part of one unit
// inside one work item).
struct SegDesc {
    int out_row;     // first row of the unit's G output rows: b*q_heads + head*G
    int uid;         // unit index over both classes: the ticket index
    int complete;    // the segment is the whole unit: normalise and write out
    int pslot;       // partial record the segment goes to otherwise
    int stop;        // no more segments: the epilogue warps leave
    int pad[3];
};

// What the producer tells the consumer warps about the next segment: they never look anything up in
// the schedule themselves (a look-up costs about a microsecond, and while the consumers sit in one at
// the start of a segment no stage is released: for a unit of two tiles that was as long as its tiles).
struct SegInfo {
    int item;              // the work item (it names the partial record); -1: no more work
    int x;                 // flat tile of the segment's first tile
    int seg_tiles;         // tiles of the segment in the schedule
    int uid, tile, band;   // the unit, the segment's first tile inside it, the band
    int tiles, len;        // tiles and valid rows of the unit
    int qrow, head, layer; // where its query and output rows are; its KV head; its layer (paged whole step)
    int pad;
};
constexpr int kSegRing = 8;  // segment descriptors in flight between producer and consumers

// Shared-memory carve-up (dynamic shared memory, base aligned to 1024 bytes for the swizzle).
template <int D, int NG>
struct Smem {
    static constexpr int kWarps = NG * kGroupWarps;         // consumer warps
    static constexpr int kThreads = (kWarps + 2 + kEpilogueWarps) * 32;
    static constexpr int kTileBytes = kTile * D * 2;        // one K (or V) tile
    static constexpr int kTilePairBytes = 2 * kTileBytes;   // K tile then V tile
    // a stage: K tile, V tile, then the G query rows of the tile's unit (filled for the first NG
    // tiles of a segment), padded so that the next stage starts on a 1024-byte boundary again
    // (8-bit pages: a stage is TWO consecutive 16 KB pages of a unit, tiles 2p and 2p + 1, each K codes
    // then V codes transposed: the per-stage costs are then paid per 128 tokens)
    __host__ __device__ static constexpr int tile_pair_bytes(int /*mode*/) { return kTilePairBytes; }
    __host__ __device__ static constexpr int stage_bytes(int group, int mode = kModePlain)
    {
        return tile_pair_bytes(mode) + (group * D * 2 + 1023) / 1024 * 1024;
    }
    static constexpr int kMergeStride = D + kMergePad;      // floats per head row
    static constexpr int kStatFloats = 2 * kWarps * kMaxGroup;
    static constexpr int kBarriers = 2 * 8 + 2 * kSegRing + 2 + 2 * kMergeBuffers + 2;  // the last two: page look-ups
    __host__ __device__ static constexpr int merge_floats(int group) { return kWarps * group * kMergeStride; }
    // one hand-off buffer: merge rows, per-warp max and sum, segment descriptor
    __host__ __device__ static constexpr int buffer_bytes(int group)
    {
        return merge_floats(group) * 4 + kStatFloats * 4 + 32;
    }
    // paged cache only: the page-table entries of the segment being streamed, the PagedArgs
    static constexpr int kPagedBytes = (kMaxSeqPages + 4) * 4 + (int)((sizeof(PagedArgs) + 15) / 16 * 16) + kMaxStepHeads;
    // whole-step launches only: the StepArgs and the KV head of every slot of every layer
    static constexpr int kStepBytes = (int)((sizeof(StepArgs) + 15) / 16 * 16) + kMaxStepHeads;
    __host__ __device__ static constexpr size_t bytes(int stages, int group, int mode = kModePlain)
    {
        return (size_t)stages * stage_bytes(group, mode) + (size_t)kMergeBuffers * buffer_bytes(group) + kBarriers * 8 +
               kSegRing * sizeof(SegInfo) /*segment descriptors*/ + 16 /*claim slot, flags*/ +
               kMaxPend * 8 /*partial segments without a ticket*/ +
               kMaxTodo * 8 /*units to merge*/ + kMaxTodo * (kMaxRounds + 2) * 8 /*their partial lists*/ +
               (sizeof(DecodeArgs) + 15) / 16 * 16 + (mode == kModePaged || mode == kModePagedFp8 ? kPagedBytes : 0) +
               (mode == kModeStep ? kStepBytes : 0);
    }
};

// Merge of split units.  `units` lists (unit, first output row) of n units whose partial records
// are all in memory, `lists` their records as (first record, count) per band; thread t of nt
// cooperating threads takes 4-float pieces of their G x D output rows.  The records of a unit are
// merged in a fixed order (band by band, item by item), 16 at a time -- all loads of a batch first,
// so a typical unit costs one trip to the L2 -- and the arithmetic does not depend on nt, so the
// result does not depend on who merges or when.  `dry`: everything but the stores -- run once by
// the idle epilogue warps at kernel start so that the instructions are in the SM's instruction
// cache when the merges at the end of the stream need them.  The caller orders the call after the
// writes to `units` and `lists`.
// (Everything comes by value or from shared memory: a reference to kernel parameters would turn
// every use into a slow generic load inside this non-inlined function.)
// MIXED (Eq. 1 of the paper): `units` lists (batch row, head) pairs; entries 0 .. R of a pair's list
// are the records of its first unit -- the tokens between the sink and the window --, entry
// kMaxRounds + 1 those of its local unit (sink and window).  No token is read twice: the full branch
// of Eq. 1 is the merge of ALL the pair's records, the local branch the merge of the local unit's, and
// the rows get gate * full + (1 - gate) * local, written once: no clearing, no atomics, and the
// result does not depend on which unit finished first.
constexpr int kListStride = kMaxRounds + 2;  // (first record, count) per band, then the local unit's (MIXED)
template <int D>
__device__ __noinline__ void merge_units_plain(const float* partials, float* out, int G, int R, const int2* units,
                                         const int2* lists, int n, int t, int nt, bool dry,
                                         unsigned long long* stamp, const float* alpha, int U, int q_heads, int out_bf16)
{
    constexpr int D4 = D / 4, CH = 16, NB = kListStride;
    const int E = G * D4;
    const int PF = partial_floats(D, G), PH = partial_head_floats(G);
    __threadfence();
    if (stamp && t == 0) stamp[0] = global_timer_ns();
    const bool wide = nt >= E;                  // enough threads for one piece each, of nt / E units at a time
    const int unit_lanes = wide ? nt / E : 1;
    const int ul = wide ? t / E : 0;
    if (ul < unit_lanes) {
        for (int j = ul; j < n; j += unit_lanes) {
            const int2* li = lists + j * NB;
            for (int e = wide ? t - ul * E : t; e < E; e += wide ? E : nt) {
                const int g = e / D4;
                float4 res = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 1
                for (int part = 0; part < (1); ++part) {  // the full unit's records, then the local unit's
                const int b0 = part ? NB - 1 : 0, b1 = part ? NB : R + 1;
                int F = 0;
                for (int r = b0; r < b1; ++r) F += li[r].y;
                float M = kNegBig, L = 0.f;
                float4 O = make_float4(0.f, 0.f, 0.f, 0.f);
                int band = b0, off = 0;  // the record with merge index c0 is record `off` of band `band`
                for (int c0 = 0; c0 < F; c0 += CH) {
                    float mm[CH], ll[CH];
                    float4 oo[CH];
#pragma unroll
                    for (int c = 0; c < CH; ++c) {
                        const bool on = c0 + c < F;
                        if (on)
                            while (off >= li[band].y) {
                                off -= li[band].y;
                                ++band;
                            }
                        const float* pc = partials + (size_t)(on ? li[band].x + off : 0) * PF;
                        mm[c] = on ? __ldcg(pc + g) : kNegBig;
                        ll[c] = on ? __ldcg(pc + G + g) : 0.f;
                        oo[c] = on ? __ldcg(reinterpret_cast<const float4*>(pc + PH) + e) : make_float4(0.f, 0.f, 0.f, 0.f);
                        ++off;
                    }
                    float Mc = M;
#pragma unroll
                    for (int c = 0; c < CH; ++c) Mc = fmaxf(Mc, mm[c]);
                    if (stamp && t == 0 && j == ul && c0 == 0) stamp[2] = global_timer_ns();
                    const float keep = exp2f(M - Mc);
                    L *= keep;
                    O.x *= keep;
                    O.y *= keep;
                    O.z *= keep;
                    O.w *= keep;
#pragma unroll
                    for (int c = 0; c < CH; ++c) {
                        const float w = exp2f(mm[c] - Mc);
                        L += ll[c] * w;
                        O.x += oo[c].x * w;
                        O.y += oo[c].y * w;
                        O.z += oo[c].z * w;
                        O.w += oo[c].w * w;
                    }
                    M = Mc;
                }
                if (stamp && t == 0 && j == ul) stamp[3] = global_timer_ns();
                float inv = 1.f / L;
                if (false) {
                    const float gate = __ldg(alpha + (units[j].y % q_heads) / G);
                    inv *= part ? 1.f - gate : gate;
                }
                res.x += O.x * inv;
                res.y += O.y * inv;
                res.z += O.z * inv;
                res.w += O.w * inv;
                }
                if (!dry) {
                    if (out_bf16)
                        *reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(out) + (size_t)units[j].y * D + e * 4) =
                            make_uint2(pack_bf16(res.x, res.y), pack_bf16(res.z, res.w));
                    else
                        *reinterpret_cast<float4*>(out + (size_t)units[j].y * D + e * 4) = res;
                }
            }
        }
    }
}

// Mixed attention (see above): one pass over all records of a pair, the local unit's also into a second state.
template <int D>
__device__ __noinline__ void merge_units_mixed(const float* partials, float* out, int G, int R, const int2* units,
                                         const int2* lists, int n, int t, int nt, bool dry,
                                         unsigned long long* stamp, const float* alpha, int U, int q_heads, int out_bf16)
{
    constexpr int D4 = D / 4, CH = 16, NB = kListStride;
    constexpr bool MIXED = true;
    const int E = G * D4;
    const int PF = partial_floats(D, G), PH = partial_head_floats(G);
    __threadfence();
    if (stamp && t == 0) stamp[0] = global_timer_ns();
    const bool wide = nt >= E;                  // enough threads for one piece each, of nt / E units at a time
    const int unit_lanes = wide ? nt / E : 1;
    const int ul = wide ? t / E : 0;
    if (ul < unit_lanes) {
        for (int j = ul; j < n; j += unit_lanes) {
            const int2* li = lists + j * NB;
            for (int e = wide ? t - ul * E : t; e < E; e += wide ? E : nt) {
                const int g = e / D4;
                // MIXED: all records of the pair make the full branch (list entries R + 1 .. NB - 2 are empty);
                // the local unit's, which come last, also go into a second state: one pass, one trip
                const int b1 = MIXED ? NB : R + 1;
                int F = 0;
                for (int r = 0; r < b1; ++r) F += li[r].y;
                const int first_local = MIXED ? F - li[NB - 1].y : F;
                float M = kNegBig, L = 0.f, M2 = kNegBig, L2 = 0.f;
                float4 O = make_float4(0.f, 0.f, 0.f, 0.f), O2 = make_float4(0.f, 0.f, 0.f, 0.f);
                int band = 0, off = 0;  // the record with merge index c0 is record `off` of band `band`
                for (int c0 = 0; c0 < F; c0 += CH) {
                    float mm[CH], ll[CH];
                    float4 oo[CH];
#pragma unroll
                    for (int c = 0; c < CH; ++c) {
                        const bool on = c0 + c < F;
                        if (on)
                            while (off >= li[band].y) {
                                off -= li[band].y;
                                ++band;
                            }
                        const float* pc = partials + (size_t)(on ? li[band].x + off : 0) * PF;
                        mm[c] = on ? __ldcg(pc + g) : kNegBig;
                        ll[c] = on ? __ldcg(pc + G + g) : 0.f;
                        oo[c] = on ? __ldcg(reinterpret_cast<const float4*>(pc + PH) + e) : make_float4(0.f, 0.f, 0.f, 0.f);
                        ++off;
                    }
                    float Mc = M;
#pragma unroll
                    for (int c = 0; c < CH; ++c) Mc = fmaxf(Mc, mm[c]);
                    if (stamp && t == 0 && j == ul && c0 == 0) stamp[2] = global_timer_ns();
                    const float keep = exp2f(M - Mc);
                    L *= keep;
                    O.x *= keep;
                    O.y *= keep;
                    O.z *= keep;
                    O.w *= keep;
#pragma unroll
                    for (int c = 0; c < CH; ++c) {
                        const float w = exp2f(mm[c] - Mc);
                        L += ll[c] * w;
                        O.x += oo[c].x * w;
                        O.y += oo[c].y * w;
                        O.z += oo[c].z * w;
                        O.w += oo[c].w * w;
                    }
                    M = Mc;
                    if (MIXED && c0 + CH > first_local) {  // the batch holds records of the local unit
                        float Mc2 = M2;
#pragma unroll
                        for (int c = 0; c < CH; ++c)
                            if (c0 + c >= first_local) Mc2 = fmaxf(Mc2, mm[c]);
                        const float keep2 = exp2f(M2 - Mc2);
                        L2 *= keep2;
                        O2.x *= keep2;
                        O2.y *= keep2;
                        O2.z *= keep2;
                        O2.w *= keep2;
#pragma unroll
                        for (int c = 0; c < CH; ++c)
                            if (c0 + c >= first_local) {
                                const float w = exp2f(mm[c] - Mc2);
                                L2 += ll[c] * w;
                                O2.x += oo[c].x * w;
                                O2.y += oo[c].y * w;
                                O2.z += oo[c].z * w;
                                O2.w += oo[c].w * w;
                            }
                        M2 = Mc2;
                    }
                }
                if (stamp && t == 0 && j == ul) stamp[3] = global_timer_ns();
                float inv = 1.f / L;
                float4 res;
                if (MIXED) {
                    const float gate = __ldg(alpha + (units[j].y % q_heads) / G);
                    inv *= gate;
                    const float inv2 = (1.f - gate) / L2;
                    res = make_float4(O.x * inv + O2.x * inv2, O.y * inv + O2.y * inv2, O.z * inv + O2.z * inv2,
                                      O.w * inv + O2.w * inv2);
                } else {
                    res = make_float4(O.x * inv, O.y * inv, O.z * inv, O.w * inv);
                }
                if (!dry) {
                    if (out_bf16)
                        *reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(out) + (size_t)units[j].y * D + e * 4) =
                            make_uint2(pack_bf16(res.x, res.y), pack_bf16(res.z, res.w));
                    else
                        *reinterpret_cast<float4*>(out + (size_t)units[j].y * D + e * 4) = res;
                }
            }
        }
    }
}

template <int D, bool MIXED>
__device__ __forceinline__ void merge_units(const float* partials, float* out, int G, int R, const int2* units,
                                            const int2* lists, int n, int t, int nt, bool dry,
                                            unsigned long long* stamp, const float* alpha, int U, int q_heads, int out_bf16)
{
    if constexpr (MIXED) merge_units_mixed<D>(partials, out, G, R, units, lists, n, t, nt, dry, stamp, alpha, U, q_heads, out_bf16);
    else merge_units_plain<D>(partials, out, G, R, units, lists, n, t, nt, dry, stamp, alpha, U, q_heads, out_bf16);
}

// ---------------------------------------------------------------------------------------------
// The kernel.  Warp roles: 0 .. 4*NG-1 consumers (group = warp / 4); then one producer warp (TMA);
// one claim warp (fetches the next work item from the global counter while the producer streams the
// current one, so no memory round trip ever sits in the producer's path); kEpilogueWarps epilogue
// warps (merge the consumer warps' states of a finished segment, write the output or the partial,
// run the ticket and the merge of split units) so that the consumer warps go straight on to the
// next segment.  All hand-offs are mbarrier rings in shared memory.
//
// Slot i % stages of the tile ring holds the i-th slot the CTA issues; the slot of flat tile x
// always has i = x (mod NG), so tile x is consumed by group x % NG whatever the CTA did before
// (results do not depend on which CTA claimed which item) and a stage is always consumed by the
// same group (stages is a multiple of NG).  Where an item starts on the wrong residue the producer
// issues an empty slot first.
//
// MIXED: the mixed attention of Eq. 1, every row read once.  The first class of units covers the rows
// between sink and window of every (batch row, head), the second class holds its LOCAL unit over the
// sink and window rows; tiles start at whatever row the range starts (a TMA box may start at any row)
// and are masked past their valid rows.  Every segment of either unit leaves a partial record; the
// pair's ticket counts the records of both, and whoever delivers the last one merges them -- all
// records for the full branch, the local unit's for the local branch -- and writes
// gate * full + (1 - gate) * local once.
//
// kModeStep: a whole decode step.  The full units of all layers are one list and so are the compressed
// units (every layer holds the same number of tokens); a unit's layer, rows, query and output rows are
// looked up in the StepArgs.  Everything else is the lock-step kernel.
//
// kModePaged: the paged cache.  Units keep the uniform layout (every full unit is given the tiles of
// the longest sequence); producer and consumers both leave out a unit's tiles past its own length and
// realign the slot counter at every segment, and the producer looks a full unit's rows up in the
// sequence's page table, whose entries for a segment it fetches with one bulk copy.
struct NoPagedArgs {};
template <int MODE>
struct ExtraArgs {
    typedef NoPagedArgs type;
};
template <>
struct ExtraArgs<kModePaged> {
    typedef PagedArgs type;
};
template <>
struct ExtraArgs<kModePagedFp8> {
    typedef PagedFp8Args type;  // starts with a PagedArgs
};
template <>
struct ExtraArgs<kModeStep> {
    typedef StepArgs type;
};

template <int D, int NG, int MODE>
__global__ void __launch_bounds__(Smem<D, NG>::kThreads, 1)
decode_kernel(const __grid_constant__ DecodeArgs args, const __grid_constant__ CUtensorMap tmap, const int stages,
              const __grid_constant__ typename ExtraArgs<MODE>::type extra)
{
    constexpr bool MIXED = MODE == kModeMixed;
    constexpr bool PAGED = MODE == kModePaged || MODE == kModePagedFp8;
    constexpr bool FP8 = MODE == kModePagedFp8;  // pages and rings hold E4M3 codes (head_dim 128 only)
    constexpr bool STEP = MODE == kModeStep;
    using S = Smem<D, NG>;
    constexpr int KS = D / 16;  // k-steps of Q.K^T; also 16-row slabs of O^T
    constexpr int MS = S::kMergeStride;
    extern __shared__ __align__(1024) uint8_t smem[];
    const int G = args.group;
    uint8_t* stage_base = smem;
    const int stage_bytes = S::stage_bytes(G, MODE);
    constexpr int kPairBytes = S::tile_pair_bytes(MODE);  // the query rows of a stage follow its K/V data
    uint8_t* buffers = smem + (size_t)stages * stage_bytes;
    const int buffer_bytes = S::buffer_bytes(G);
    uint64_t* full_bar = reinterpret_cast<uint64_t*>(buffers + (size_t)kMergeBuffers * buffer_bytes);
    uint64_t* empty_bar = full_bar + 8;
    uint64_t* seg_full = empty_bar + 8;
    uint64_t* seg_empty = seg_full + kSegRing;
    uint64_t* claim_full = seg_empty + kSegRing;
    uint64_t* claim_empty = claim_full + 1;
    uint64_t* ep_full = claim_empty + 1;
    uint64_t* ep_empty = ep_full + kMergeBuffers;
    uint64_t* page_bar = ep_empty + kMergeBuffers;  // [2], the second one unused
    SegInfo* seg_desc = reinterpret_cast<SegInfo*>(page_bar + 2);
    volatile int* claim_slot = reinterpret_cast<volatile int*>(seg_desc + kSegRing);
    volatile int* ep_flag = claim_slot + 1;
    volatile int* s_abort = claim_slot + 2;
    int2* pend = reinterpret_cast<int2*>(const_cast<int*>(claim_slot) + 4);  // [kMaxPend] (unit, first output row)
    int2* todo = pend + kMaxPend;                                           // [kMaxTodo] units whose partials are all in
    int2* lists = todo + kMaxTodo;                                          // scratch of merge_units
    int* todo_count = const_cast<int*>(claim_slot) + 3;
    // The arguments, copied to shared memory: the schedule and the head order are looked up with
    // run-time indices, which is slow on kernel parameters and cheap here.
    DecodeArgs* s_args = reinterpret_cast<DecodeArgs*>(lists + kMaxTodo * kListStride);
    const DecodeArgs& a = *s_args;
    // paged cache: lengths and request slots of the batch, then the page ids of one segment
    PagedArgs* s_paged = reinterpret_cast<PagedArgs*>(reinterpret_cast<uint8_t*>(s_args) + (sizeof(DecodeArgs) + 15) / 16 * 16);
    int* s_pages = reinterpret_cast<int*>(reinterpret_cast<uint8_t*>(s_paged) + (sizeof(PagedArgs) + 15) / 16 * 16);
    const PagedArgs* pg = PAGED ? s_paged : nullptr;
    // whole-step launch: the layer tables and the KV head of every slot, at the same place
    const StepArgs* stp = STEP ? reinterpret_cast<const StepArgs*>(s_paged) : nullptr;
    unsigned char* s_heads = PAGED ? reinterpret_cast<unsigned char*>(s_pages + kMaxSeqPages + 4)
                                   : reinterpret_cast<unsigned char*>(s_paged) + (sizeof(StepArgs) + 15) / 16 * 16;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const Schedule& sc = a.sched;
    const bool trace = args.trace_on != 0;
    unsigned long long* my_trace = args.trace + (size_t)blockIdx.x * kTraceWords;
    if (trace && tid == 0) my_trace[0] = global_timer_ns();
    // Overlapped launches (the layers of one decode step): the next layer's kernel is scheduled as SMs
    // become free and uses the other copy of the scratch memory, so it touches nothing this one uses.
    // A launch lets its successor start (launch_dependents) only once its own predecessor has completed:
    // two launches that share a scratch copy are then never in flight together.
    //   dep_wait == 0: an ordinary launch; its predecessor completed before it started.
    //   dep_wait == 1: the step's first decode launch, which may run beside the step's append launch: it
    //     fetches and processes tiles that hold only older tokens, waits (grid_dep_wait) before it touches
    //     anything else, and only then lets the next layer start.
    //   dep_wait == 2: any later launch of the step, which may run beside its predecessor: an otherwise
    //     idle thread of every CTA waits for the predecessor and only then lets the next launch start.
    //   dep_wait == 3: a per-layer call that may start before the kernel that produces its q (and before
    //     the append of this step's token) has completed: the producer fetches K/V tiles of older tokens
    //     -- as many as the tile ring holds -- and waits before it fetches the query rows, the newest
    //     tile or a ring; claims, tickets, partials and results come after a wait as well.  The next
    //     kernel of the stream may start at once (it waits for this one itself before it reads `out`).
    if (tid == 0 && (!args.dep_wait || args.dep_wait == 3)) grid_dep_launch();

    if ((smem_u32(smem) & 1023u) != 0) {  // uniform over the CTA: nobody has touched a barrier yet
        if (tid == 0) atomicCAS(args.status, kStatusOk, kStatusSmemMisaligned);
        return;
    }
    for (int i = tid; i < (int)(sizeof(DecodeArgs) / sizeof(int)); i += blockDim.x)
        reinterpret_cast<int*>(s_args)[i] = reinterpret_cast<const int*>(&args)[i];
    if constexpr (PAGED) {
        // only what the launch uses: reading kernel parameters with a per-thread index is slow, and the
        // per-sequence and per-layer arrays are sized for 512 sequences and 128 layers
        const PagedArgs& ex = *reinterpret_cast<const PagedArgs*>(&extra);
        const bool whole = ex.step.n_layers > 1;
        const int n_seq = whole ? ex.step.batch : args.batch;
        auto copy_ints = [&](size_t first_byte, size_t end_byte) {
            for (int i = (int)(first_byte / 4) + tid; i < (int)((end_byte + 3) / 4); i += blockDim.x)
                reinterpret_cast<int*>(s_paged)[i] = reinterpret_cast<const int*>(&extra)[i];
        };
        copy_ints(0, offsetof(PagedArgs, seq_len) + (size_t)n_seq * sizeof(int));
        copy_ints(offsetof(PagedArgs, seq_slot), offsetof(PagedArgs, seq_slot) + (size_t)n_seq * sizeof(unsigned short));
        copy_ints(offsetof(PagedArgs, step), offsetof(PagedArgs, step) + offsetof(StepArgs, full_base));
        if (whole) {
            const size_t L = (size_t)ex.step.n_layers;
            const size_t st = offsetof(PagedArgs, step);
            copy_ints(st + offsetof(StepArgs, full_base), st + offsetof(StepArgs, full_base) + (L + 1) * 4);
            copy_ints(st + offsetof(StepArgs, comp_base), st + offsetof(StepArgs, comp_base) + (L + 1) * 4);
            copy_ints(st + offsetof(StepArgs, full_row0), st + offsetof(StepArgs, full_row0) + L * 4);
            copy_ints(st + offsetof(StepArgs, comp_row0), st + offsetof(StepArgs, comp_row0) + L * 4);
            copy_ints(offsetof(PagedArgs, scales), offsetof(PagedArgs, scales) + sizeof(const float*));
            copy_ints(offsetof(PagedArgs, page0_8_of), offsetof(PagedArgs, page0_8_of) + L * 4);
            copy_ints(offsetof(PagedArgs, ring0_8_of), offsetof(PagedArgs, ring0_8_of) + L * 4);
            // the KV head of every slot of every layer (written at cache creation)
            for (int i = tid; i < ex.step.n_layers * ex.step.kv_heads; i += blockDim.x)
                s_heads[i] = (unsigned char)__ldg(ex.step.head_of_slot + i);
        }
    }
    if constexpr (STEP) {
        // (the per-layer arrays are sized for 128 layers: only the layers of the launch are copied)
        const int L = extra.n_layers;
        auto copy_ints = [&](size_t first_byte, size_t end_byte) {
            for (int i = (int)(first_byte / 4) + tid; i < (int)((end_byte + 3) / 4); i += blockDim.x)
                reinterpret_cast<int*>(s_paged)[i] = reinterpret_cast<const int*>(&extra)[i];
        };
        copy_ints(0, offsetof(StepArgs, full_base) + (size_t)(L + 1) * 4);
        copy_ints(offsetof(StepArgs, comp_base), offsetof(StepArgs, comp_base) + (size_t)(L + 1) * 4);
        copy_ints(offsetof(StepArgs, full_row0), offsetof(StepArgs, full_row0) + (size_t)L * 4);
        copy_ints(offsetof(StepArgs, comp_row0), offsetof(StepArgs, comp_row0) + (size_t)L * 4);
        for (int i = tid; i < extra.n_layers * extra.kv_heads; i += blockDim.x)  // written at cache creation
            s_heads[i] = (unsigned char)__ldg(extra.head_of_slot + i);
    }
    if (tid == 0) {
        for (int s = 0; s < stages; ++s) {
            mbar_init(smem_u32(full_bar + s), 1);
            mbar_init(smem_u32(empty_bar + s), kGroupWarps);
        }
        for (int i = 0; i < kSegRing; ++i) {
            mbar_init(smem_u32(seg_full + i), 1);
            mbar_init(smem_u32(seg_empty + i), S::kWarps);
        }
        mbar_init(smem_u32(claim_full), 1);
        mbar_init(smem_u32(claim_empty), 1);
        mbar_init(smem_u32(page_bar), 1);
        for (int i = 0; i < kMergeBuffers; ++i) {
            mbar_init(smem_u32(ep_full + i), S::kWarps);
            mbar_init(smem_u32(ep_empty + i), kEpilogueWarps);
        }
        *ep_flag = 0;
        *s_abort = 0;
        *todo_count = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (trace && tid == 0) my_trace[38] = global_timer_ns();

    int issued = 0;  // producer: slots issued so far (data or empty)
    int page_lost_par = -1;  // producer, paged cache: phase of a page look-up it gave up waiting for
    if (warp < S::kWarps) {
        // ------------------------------------------------------------------ consumer warps
        const int grp = warp / kGroupWarps, wig = warp % kGroupWarps;  // tile group, 16-token slice
        const int quad = lane >> 2, tq = lane & 3;  // row inside an 8-row fragment, column pair
        const int ldm_j = lane >> 3, ldm_r = lane & 7;
        const int ldm_tok = wig * 16 + (ldm_j >> 1) * 8 + ldm_r;  // token row this lane addresses
        const int ldm_chunk = ldm_j & 1;                          // +1 16-byte chunk for odd matrices
        int cnt = 0;   // slots seen so far (mirrors the producer's `issued`)
        int st = 0, turn = 0;  // cnt % stages, cnt % NG
        uint32_t ph = 0;       // (cnt / stages) & 1
        auto next_slot = [&]() {
            ++cnt;
            if (++turn == NG) turn = 0;
            if (++st == stages) {
                st = 0;
                ph ^= 1u;
            }
        };
        int seg = 0;   // segments handed to the epilogue warps so far
        int di = 0;
        uint32_t dpar = 0;
        int n_items = 0, n_tiles = 0, n_partial = 0;  // trace counters
        unsigned long long ns_item = 0, ns_tile = 0, ns_merge = 0;
        const bool tr0 = trace && tid == 0;
        bool landed = false, alive = true;
        int last_item = -1;
        while (alive) {
            // ---- the next segment, as the producer describes it: tiles [x, x + seg_tiles) of one unit
            // (none for the stop message).  The descriptor is copied and its slot given back at once.
            if (!wait_traced(smem_u32(seg_full + di), dpar, s_abort, a.status, kStatusItemWaitTimeout, tr0, &ns_item)) break;
            const SegInfo sg = seg_desc[di];
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(seg_empty + di));
            if (++di == kSegRing) {
                di = 0;
                dpar ^= 1u;
            }
            const int item = sg.item, x = sg.x;
            if (item >= 0 && item != last_item) {
                if (tr0 && n_items < 11) my_trace[16 + n_items] = (global_timer_ns() << 16) | (unsigned long long)(item & 0xffff);
                ++n_items;
                last_item = item;
            }
            {
                UnitInfo u{};
                u.pos.uid = sg.uid;
                u.pos.tile = sg.tile;
                u.pos.band = sg.band;
                u.tiles = sg.tiles;
                u.len = sg.len;
                u.qrow = sg.qrow;
                u.head = sg.head;
                u.layer = sg.layer;
                int seg_tiles = 0;
                float m_run = kNegBig, l_run = 0.f;
                // 8-bit pages: the first product has the tokens as rows and the heads as columns, so a lane
                // keeps the running maximum and sum of heads 2tq (m_run, l_run) and 2tq + 1 (these)
                float m_run1 = kNegBig, l_run1 = 0.f;
                float acc[KS][4];
#pragma unroll
                for (int mt = 0; mt < KS; ++mt) acc[mt][0] = acc[mt][1] = acc[mt][2] = acc[mt][3] = 0.f;
                if (item >= 0) {
                    seg_tiles = sg.seg_tiles;
                    const bool local_unit = MIXED && u.pos.uid >= sc.U;
                    const bool fp8_unit = FP8;  // every unit of an 8-bit cache is pages of E4M3 codes
                    int seg_eff = seg_tiles;  // tiles of the segment that exist (the producer announces no segment without any)
                    if (PAGED) seg_eff = max(0, min(seg_tiles, (u.len + kTile - 1) / kTile - u.pos.tile));
                    // skip the empty slots the producer issued to line the slot counter up with x (a new item
                    // may start anywhere; tiles a paged unit does not have shift the counter against x)
                    for (int pad = ((x - cnt) % NG + NG) % NG; alive && pad > 0; --pad, next_slot()) {
                        if (turn != grp) continue;
                        alive = wait_bounded(smem_u32(full_bar + st), ph, s_abort, a.status, kStatusFullWaitTimeout);
                        if (alive && lane == 0) mbar_arrive(smem_u32(empty_bar + st));
                    }
                    // Q as the A operand (rows = query heads of the group, rows >= G are zero): read from
                    // the stage of this warp's first tile of the segment, where the producer put the
                    // unit's query rows
                    uint32_t qa[KS][2];
                    bool have_q = false;
                    int valid_left = u.len - u.pos.tile * kTile;  // valid rows from this tile to the unit's end
                    int step = 1;  // tiles in the slot (8-bit pages: two where the unit has an even-odd pair here)
                    for (int i = 0; alive && i < seg_eff; i += step, next_slot(), valid_left -= step * kTile) {
                        if (FP8) step = ((u.pos.tile + i) & 1) ? 1 : min(2, seg_eff - i);
                        if (turn != grp) continue;
                        alive = wait_traced(smem_u32(full_bar + st), ph, s_abort, a.status, kStatusFullWaitTimeout, tr0,
                                            &ns_tile);
                        if (!alive) break;
                        if (trace && tid == 0 && !landed) {
                            my_trace[1] = global_timer_ns();
                            landed = true;
                        }
                        int valid = min(kTile, valid_left);
                        if (local_unit) {
                            int row;
                            local_tile(a, u.pos.tile + i, row, valid);
                        }
                        if (FP8 && fp8_unit && !have_q) {
                            // the contraction index may be permuted as long as both operands agree: against
                            // codes fetched four consecutive d per lane, Q goes in as f16 with k-halves
                            // (d 4tq, 4tq+1) and (d 4tq+2, 4tq+3) of every 16
                            const __nv_bfloat16* qrow = reinterpret_cast<const __nv_bfloat16*>(
                                                            stage_base + (size_t)st * stage_bytes + kPairBytes) +
                                                        quad * D + 4 * tq;
#pragma unroll
                            for (int ks = 0; ks < KS; ++ks) {
                                const uint2 raw = quad < G ? *reinterpret_cast<const uint2*>(qrow + ks * 16) : make_uint2(0u, 0u);
                                const float2 f0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw.x));
                                const float2 f1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw.y));
                                qa[ks][0] = pack_f16(f0.x, f0.y);
                                qa[ks][1] = pack_f16(f1.x, f1.y);
                            }
                            have_q = true;
                        }
                        if (!have_q) {
                            const __nv_bfloat16* qrow = reinterpret_cast<const __nv_bfloat16*>(
                                                            stage_base + (size_t)st * stage_bytes + kPairBytes) +
                                                        quad * D + 2 * tq;
#pragma unroll
                            for (int ks = 0; ks < KS; ++ks) {
                                qa[ks][0] = quad < G ? *reinterpret_cast<const uint32_t*>(qrow + ks * 16) : 0u;
                                qa[ks][1] = quad < G ? *reinterpret_cast<const uint32_t*>(qrow + ks * 16 + 8) : 0u;
                            }
                            have_q = true;
                        }
                        if (FP8 && fp8_unit) {
                            // The slot's tiles (two where the unit has an even-odd pair here): an 8-bit page is 128
                            // rows of 128 bytes under the 128-byte swizzle, K codes [64 tokens][128], then V codes
                            // transposed [128 d][64 tokens], two d per row; an even tile's page is the first of
                            // the stage, an odd tile's the second.  The scores of both tiles go through ONE
                            // softmax update: one maximum, one correction of the accumulators per 128 tokens.
                            const int lj = lane >> 3, li = lane & 7;
                            // ldmatrix row i of token set s is token 4(i/2) + 2s + (i%2) of the warp's 16, so that
                            // this lane ends up with four consecutive tokens
                            const int ktok = wig * 16 + 4 * (li >> 1) + 2 * (lj & 1) + (li & 1);
                            const uint32_t stage0 = smem_u32(stage_base + (size_t)st * stage_bytes);
                            // K's scale joins the softmax scale
                            const float sl2 = a.scale_log2 * (pg->step.n_layers > 1 ? __ldg(pg->scales + u.layer * pg->step.kv_heads + u.head)
                                                                                    : pg->k_scale[u.head]);
                            // scores of this lane per tile: [0], [1] token row `quad` of set A, heads 2tq and 2tq+1;
                            // [2], [3] token row `quad` of set B, the same heads
                            float sc8[2][4];
                            bool active[2];
#pragma unroll
                            for (int sb = 0; sb < 2; ++sb) {
                                const int valid_sb = min(kTile, valid_left - sb * kTile);  // of this tile of the slot
                                active[sb] = sb < step && wig * 16 < valid_sb;
                                sc8[sb][0] = sc8[sb][1] = sc8[sb][2] = sc8[sb][3] = -INFINITY;
                                if (active[sb]) {
                                    const uint32_t sK = stage0 + ((u.pos.tile + i + sb) & 1) * (2 * kTile * 128);
                                    // ---- S^T = K.Q^T: the 16 tokens are the rows (set A rows 0-7, set B rows 8-15),
                                    // the query heads the 8 columns -- one MMA per 16 d, where the heads as rows
                                    // would take two, half of them padding.  All fragments of K first.
                                    float se[4] = {0.f, 0.f, 0.f, 0.f}, so[4] = {0.f, 0.f, 0.f, 0.f};
                                    uint32_t kf[KS / 2][4];
#pragma unroll
                                    for (int kp = 0; kp < KS / 2; ++kp) {
                                        const int chunk = 2 * kp + (lj >> 1);  // 16 codes along d
                                        ldmatrix_x4(sK + ktok * 128 + ((chunk ^ (ktok & 7)) << 4), kf[kp][0], kf[kp][1],
                                                    kf[kp][2], kf[kp][3]);
                                    }
#pragma unroll
                                    for (int kp = 0; kp < KS / 2; ++kp) {
                                        uint32_t a0, a1, a2, a3;
                                        e4m3x4_to_f16x2x2(kf[kp][0], a0, a2);  // set A, chunk 2kp
                                        e4m3x4_to_f16x2x2(kf[kp][1], a1, a3);  // set B, chunk 2kp
                                        mma_f16(se, a0, a1, a2, a3, qa[2 * kp][0], qa[2 * kp][1]);
                                        e4m3x4_to_f16x2x2(kf[kp][2], a0, a2);  // set A, chunk 2kp + 1
                                        e4m3x4_to_f16x2x2(kf[kp][3], a1, a3);  // set B, chunk 2kp + 1
                                        mma_f16(so, a0, a1, a2, a3, qa[2 * kp + 1][0], qa[2 * kp + 1][1]);
                                    }
                                    sc8[sb][0] = (se[0] + so[0]) * sl2;
                                    sc8[sb][1] = (se[1] + so[1]) * sl2;
                                    sc8[sb][2] = (se[2] + so[2]) * sl2;
                                    sc8[sb][3] = (se[3] + so[3]) * sl2;
                                    // row `quad` of set A is token 4(quad/2) + quad%2 of the warp's 16, of set B two on
                                    const int tokA = wig * 16 + 4 * (quad >> 1) + (quad & 1);
                                    if (tokA >= valid_sb) sc8[sb][0] = sc8[sb][1] = -INFINITY;
                                    if (tokA + 2 >= valid_sb) sc8[sb][2] = sc8[sb][3] = -INFINITY;
                                }
                            }
                            if (active[0] || active[1]) {  // uniform over the warp
                                // ---- one online-softmax update for the slot (log2 domain): the maxima of heads 2tq
                                // and 2tq+1 over this lane's tokens, then over the quads
                                float mx0 = fmaxf(fmaxf(sc8[0][0], sc8[0][2]), fmaxf(sc8[1][0], sc8[1][2]));
                                float mx1 = fmaxf(fmaxf(sc8[0][1], sc8[0][3]), fmaxf(sc8[1][1], sc8[1][3]));
#pragma unroll
                                for (int o = 4; o < 32; o <<= 1) {
                                    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, o));
                                    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, o));
                                }
                                const float mn0 = fmaxf(m_run, mx0), mn1 = fmaxf(m_run1, mx1);
                                const float ca = exp2f(m_run - mn0), cb = exp2f(m_run1 - mn1);
                                float pr[2][4];
                                float ps0 = 0.f, ps1 = 0.f;
#pragma unroll
                                for (int sb = 0; sb < 2; ++sb) {
                                    pr[sb][0] = exp2f(sc8[sb][0] - mn0);
                                    pr[sb][1] = exp2f(sc8[sb][1] - mn1);
                                    pr[sb][2] = exp2f(sc8[sb][2] - mn0);
                                    pr[sb][3] = exp2f(sc8[sb][3] - mn1);
                                    ps0 += pr[sb][0] + pr[sb][2];
                                    ps1 += pr[sb][1] + pr[sb][3];
                                }
                                l_run = l_run * ca + ps0;
                                l_run1 = l_run1 * cb + ps1;
                                m_run = mn0;
                                m_run1 = mn1;
                                // O^T columns of this lane are heads 2tq and 2tq+1: its own corrections
#pragma unroll
                                for (int mt = 0; mt < KS; ++mt) {
                                    acc[mt][0] *= ca;
                                    acc[mt][1] *= cb;
                                    acc[mt][2] *= ca;
                                    acc[mt][3] *= cb;
                                }
                                // ---- O^T[d][head] += V^T[d][tok] . P^T[tok][head], tile by tile: V^T rows come
                                // straight out of the transposed page, four consecutive tokens per lane
#pragma unroll
                                for (int sb = 0; sb < 2; ++sb) {
                                    if (!active[sb]) continue;
                                    const uint32_t sV = stage0 + ((u.pos.tile + i + sb) & 1) * (2 * kTile * 128) + kTile * 128;
                                    // P is held tokens x heads; the second product wants it heads x tokens
                                    const uint32_t pb0 = movmatrix_trans(pack_f16(pr[sb][0], pr[sb][1]));
                                    const uint32_t pb1 = movmatrix_trans(pack_f16(pr[sb][2], pr[sb][3]));
                                    uint32_t vf[KS / 2][4];
#pragma unroll
                                    for (int mp = 0; mp < KS / 2; ++mp) {
                                        // row d of the transposed block is half of 128-byte row d / 2 of the page
                                        const int vd = 16 * (2 * mp + (lj >> 1)) + 8 * (lj & 1) + li, vr = vd >> 1;
                                        ldmatrix_x4(sV + vr * 128 + ((((vd & 1) * 4 + wig) ^ (vr & 7)) << 4), vf[mp][0], vf[mp][1],
                                                    vf[mp][2], vf[mp][3]);
                                    }
#pragma unroll
                                    for (int mp = 0; mp < KS / 2; ++mp) {
                                        uint32_t a0, a1, a2, a3;
                                        e4m3x4_to_f16x2x2(vf[mp][0], a0, a2);
                                        e4m3x4_to_f16x2x2(vf[mp][1], a1, a3);
                                        mma_f16(acc[2 * mp], a0, a1, a2, a3, pb0, pb1);
                                        e4m3x4_to_f16x2x2(vf[mp][2], a0, a2);
                                        e4m3x4_to_f16x2x2(vf[mp][3], a1, a3);
                                        mma_f16(acc[2 * mp + 1], a0, a1, a2, a3, pb0, pb1);
                                    }
                                }
                            }
                        } else if (wig * 16 < valid) {
                            const uint32_t sK = smem_u32(stage_base + (size_t)st * stage_bytes);
                            const uint32_t sV = sK + S::kTileBytes;
                            // ---- S = Q.K^T for this warp's 16 tokens (two 8-token column blocks)
                            float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
                            float s2[4] = {0.f, 0.f, 0.f, 0.f}, s3[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                            for (int ks = 0; ks < KS; ++ks) {
                                const int chunk = ks * 2 + ldm_chunk;  // 16-byte chunk along d
                                const uint32_t addr = sK + tile_offset<D>(ldm_tok, chunk);
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
                            float sc4[4];
                            sc4[0] = (s0[0] + s2[0]) * a.scale_log2;
                            sc4[1] = (s0[1] + s2[1]) * a.scale_log2;
                            sc4[2] = (s1[0] + s3[0]) * a.scale_log2;
                            sc4[3] = (s1[1] + s3[1]) * a.scale_log2;
                            const int tok0 = wig * 16 + 2 * tq;
                            if (tok0 >= valid) sc4[0] = -INFINITY;
                            if (tok0 + 1 >= valid) sc4[1] = -INFINITY;
                            if (tok0 + 8 >= valid) sc4[2] = -INFINITY;
                            if (tok0 + 9 >= valid) sc4[3] = -INFINITY;
                            // ---- online softmax (log2 domain)
                            float mx = fmaxf(fmaxf(sc4[0], sc4[1]), fmaxf(sc4[2], sc4[3]));
                            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
                            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
                            const float m_new = fmaxf(m_run, mx);
                            const float corr = exp2f(m_run - m_new);
                            const float p0 = exp2f(sc4[0] - m_new), p1 = exp2f(sc4[1] - m_new);
                            const float p2 = exp2f(sc4[2] - m_new), p3 = exp2f(sc4[3] - m_new);
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
                                const uint32_t addr = sV + tile_offset<D>(ldm_tok, chunk);
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
                        if (lane == 0) mbar_arrive(smem_u32(empty_bar + st));
                    }
                    if (!alive) break;
                }

                // ---- hand the warp's state (or the stop message) to the epilogue warps
                const int bi = seg % kMergeBuffers;
                alive = wait_traced(smem_u32(ep_empty + bi), ((uint32_t)(seg / kMergeBuffers) & 1u) ^ 1u, s_abort,
                                    a.status, kStatusMergeWaitTimeout, tr0, &ns_merge);
                if (!alive) break;
                uint8_t* buf = buffers + (size_t)bi * buffer_bytes;
                float* merge = reinterpret_cast<float*>(buf);
                float* stat_m = merge + S::merge_floats(G);
                float* stat_l = stat_m + S::kWarps * kMaxGroup;
                if (FP8 && item >= 0) {  // the rows were value(code): V's scale goes in here
                    const float vs = pg->step.n_layers > 1
                                         ? __ldg(pg->scales + (pg->step.n_layers + u.layer) * pg->step.kv_heads + u.head)
                                         : pg->v_scale[u.head];
#pragma unroll
                    for (int mt = 0; mt < KS; ++mt) {
                        acc[mt][0] *= vs;
                        acc[mt][1] *= vs;
                        acc[mt][2] *= vs;
                        acc[mt][3] *= vs;
                    }
                }
                if (FP8 && item >= 0) {  // sums over the lanes that hold the other tokens (same tq, other quads)
#pragma unroll
                    for (int o = 4; o < 32; o <<= 1) {
                        l_run += __shfl_xor_sync(0xffffffffu, l_run, o);
                        l_run1 += __shfl_xor_sync(0xffffffffu, l_run1, o);
                    }
                    if (quad == 0) {
                        stat_m[warp * kMaxGroup + 2 * tq] = m_run;
                        stat_l[warp * kMaxGroup + 2 * tq] = l_run;
                        stat_m[warp * kMaxGroup + 2 * tq + 1] = m_run1;
                        stat_l[warp * kMaxGroup + 2 * tq + 1] = l_run1;
                    }
                } else if (item >= 0) {
                    l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
                    l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
                    if (tq == 0) {
                        stat_m[warp * kMaxGroup + quad] = m_run;
                        stat_l[warp * kMaxGroup + quad] = l_run;
                    }
                }
                if (item >= 0) {
                    float* mw = merge + (size_t)warp * G * MS;
                    const int h0 = 2 * tq, h1 = 2 * tq + 1;
#pragma unroll
                    for (int mt = 0; mt < KS; ++mt) {
                        const int d0 = mt * 16 + quad;
                        if (h0 < G) {
                            mw[h0 * MS + d0] = acc[mt][0];
                            mw[h0 * MS + d0 + 8] = acc[mt][2];
                        }
                        if (h1 < G) {
                            mw[h1 * MS + d0] = acc[mt][1];
                            mw[h1 * MS + d0 + 8] = acc[mt][3];
                        }
                    }
                }
                if (warp == 0 && lane == 0) {
                    SegDesc* sd = reinterpret_cast<SegDesc*>(stat_l + S::kWarps * kMaxGroup);
                    // the whole unit (paged cache: all of its tiles that exist) in one segment
                    // (mixed attention: a pair's rows are written once both of its units are in, so every
                    // segment goes the way of the partial records)
                    const bool complete = !MIXED && u.pos.tile == 0 &&
                                          (PAGED ? seg_tiles >= (u.len + kTile - 1) / kTile : seg_tiles == u.tiles);
                    sd->out_row = u.qrow * a.q_heads + u.head * G;
                    sd->uid = u.pos.uid;
                    sd->complete = complete ? 1 : 0;
                    sd->pslot = item < 0 ? 0 : partial_slot(sc, u.pos.band, item, u.pos.uid);
                    sd->stop = item < 0 ? 1 : 0;
                    n_tiles += seg_tiles;
                    if (item >= 0 && !complete) ++n_partial;
                    if (trace) my_trace[2] = global_timer_ns();
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(ep_full + bi));  // release: the warp's rows are visible
                ++seg;
                if (item < 0) {
                    alive = false;  // the stop message was the last thing to do
                    break;
                }
            }
        }
        if (trace && tid == 0) {
            my_trace[4] = (unsigned long long)n_items;
            my_trace[5] = (unsigned long long)n_tiles;
            my_trace[6] = (unsigned long long)n_partial;
            my_trace[8] = ns_item;
            my_trace[9] = ns_tile;
            my_trace[10] = ns_merge;
        }
    } else if (warp == S::kWarps) {
        // ------------------------------------------------------------------ producer warp
        if (lane == 0) {
            asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap) : "memory");
            const uint64_t stream_policy = l2_evict_first_policy();
            int s = 0, di = 0;
            uint32_t par = 0, dpar = 0, cpar = 0;
            bool ok = true;
            unsigned long long ns_claim = 0, ns_ring = 0, ns_stage = 0;
            long long cy_expect = 0, cy_tma = 0, cy_q = 0, cy_item = 0, cy_seg = 0;
            const long long t_prod = clock64();
            if (trace) my_trace[39] = global_timer_ns();
            int k = blockIdx.x;  // the host launches no more CTAs than there are items
            bool synced = false;  // has waited for the kernels before this one
            uint32_t ppar = 0;    // PAGED: phase of the page look-up barrier
            const bool early = a.dep_wait == 1 || a.dep_wait == 3;  // the launch may run before its inputs are complete
            // dep_wait 3: query rows whose copy is put off until the kernel that writes them has completed
            uint32_t late_dst[8], late_bar[8];
            const __nv_bfloat16* late_src[8];
            int n_late = 0;
            auto sync_now = [&]() {
                grid_dep_wait();
                synced = true;
                for (int j = 0; j < n_late; ++j) bulk_load(late_dst[j], late_src[j], G * D * 2, late_bar[j]);
                n_late = 0;
            };
            // empty slots until the slot counter has the residue of flat tile x (tile x always goes to
            // consumer group x mod NG, whatever the CTA did before)
            auto pad_to = [&](int x) {
                for (int pad = ((x - issued) % NG + NG) % NG; ok && pad > 0; --pad) {
                    ok = wait_bounded(smem_u32(empty_bar + s), par ^ 1u, s_abort, a.status, kStatusEmptyWaitTimeout);
                    if (!ok) break;
                    mbar_arrive(smem_u32(full_bar + s));
                    ++issued;
                    if (++s == stages) {
                        s = 0;
                        par ^= 1u;
                    }
                }
            };
            // tells the consumer warps about the segment whose tiles come next (item < 0: no more work)
            auto announce = [&](int item, int x, int seg_tiles, const UnitInfo& u) {
                ok = wait_traced(smem_u32(seg_empty + di), dpar ^ 1u, s_abort, a.status, kStatusItemWaitTimeout, trace, &ns_ring);
                if (!ok) return;
                SegInfo& sg = seg_desc[di];
                sg.item = item;
                sg.x = x;
                sg.seg_tiles = seg_tiles;
                sg.uid = u.pos.uid;
                sg.tile = u.pos.tile;
                sg.band = u.pos.band;
                sg.tiles = u.tiles;
                sg.len = u.len;
                sg.qrow = u.qrow;
                sg.head = u.head;
                sg.layer = u.layer;
                mbar_arrive(smem_u32(seg_full + di));  // release: the descriptor is visible to the waiters
                if (++di == kSegRing) {
                    di = 0;
                    dpar ^= 1u;
                }
            };
            // the unit of the segment being issued; whether that segment ends where the unit's slice ends; the
            // region (prefix, band, compressed units) it lies in: its end, and first tile and width of a slice
            UnitInfo cur{};
            bool cur_slice_done = false;
            int region_end = 0, region_tile0 = 0, region_width = 0;
            int k_claim = k;  // CTA c starts with item c; the claims after that are handed items in claim_to_item's order
            while (ok && k_claim < sc.n_items) {
                const long long ti0 = trace ? clock64() : 0;
                k = claim_to_item(sc, k_claim);
                const int x0 = item_start(sc, k), x1 = item_start(sc, k + 1);
                // ask the claim warp for the next item only shortly before this one is issued in
                // full: early enough to hide the round trip, late enough that a CTA is never
                // committed to more than the tiles in its ring plus a few
                const int x_ask = max(x0, x1 - kClaimAhead);
                if (trace) cy_item += clock64() - ti0;
                int seg_left = 0, seg_idx = 0, krow = 0, vrow = 0;
                cur_slice_done = false;  // a new item starts wherever the schedule says
                int local_row0 = -1, local_next = 0;  // MIXED, inside a local unit: first row of its head, next tile
                // PAGED: tiles of the segment past the unit's own length (not issued); first pool row of the
                // full head's pages (-1: a compressed unit); page-table index of s_pages[0]; next tile
                int seg_skip = 0, paged_row0 = -1, page_base = 0, paged_tile = 0, ring_next = 0;
                int cur_tile = 0, newest_tile = -1;  // lock-step cache: the tile about to be issued, the full unit's last tile
                // a launch that also appends the step's token (DecodeArgs::new_k): the tile and the row, inside
                // the unit, that the token goes to; where its K row comes from
                int new_tile = -1, new_row = 0, new_unit_row0 = 0, new_vrows = 0;
                const __nv_bfloat16* new_src = nullptr;
                bool asked = false;
                const __nv_bfloat16* qsrc = nullptr;
                for (int x = x0; ok && x < x1; ++x) {
                    if (PAGED) {
                        if (!asked && x >= x_ask) {
                            mbar_arrive(smem_u32(claim_empty));
                            asked = true;
                        }
                    } else if (x == x_ask) {
                        mbar_arrive(smem_u32(claim_empty));
                    }
                    const long long ts0 = trace ? clock64() : 0;
                    if (seg_left == 0) {  // a new segment: where its rows are, whose query rows it needs
                        // the unit: the successor of the one before where that one's slice was issued to its
                        // end and the region goes on; looked up otherwise
                        bool stepped = false;
                        if (cur_slice_done && x < region_end) {
                            stepped = next_unit<MODE>(a, cur, pg, stp, s_heads);
                            cur.pos.tile = region_tile0;
                            cur.pos.run = region_width;
                        }
                        if (!stepped) {
                            cur = locate<MODE>(a, x, pg, stp, s_heads);
                            if (cur.pos.band < 0) {                 // the whole-unit prefix
                                region_end = sc.x0;
                                region_tile0 = 0;
                                region_width = sc.tf;
                            } else if (cur.pos.uid < sc.U) {        // a band of the full units
                                region_end = sc.base[cur.pos.band + 1];
                                region_tile0 = sc.tb[cur.pos.band];
                                region_width = sc.tb[cur.pos.band + 1] - region_tile0;
                            } else {                                // the compressed units
                                region_end = sc.T;
                                region_tile0 = 0;
                                region_width = sc.tc;
                            }
                        }
                        const UnitInfo& u = cur;
                        seg_left = min(x1 - x, u.pos.run);
                        cur_slice_done = seg_left == u.pos.run;
                        seg_idx = 0;
                        local_row0 = -1;
                        if (PAGED) {
                            const int seg_eff = max(0, min(seg_left, (u.len + kTile - 1) / kTile - u.pos.tile));
                            seg_skip = seg_left - seg_eff;
                            seg_left = seg_eff;
                            if (seg_eff == 0) {  // nothing of this unit here
                                x += seg_skip - 1;
                                continue;
                            }
                            // the step's append launch writes page-table entries and rows this launch reads:
                            // the first layer's launch waits for it before its first look-up
                            if (a.dep_wait == 1 && !synced) {
                                grid_dep_wait();
                                synced = true;
                            }
                            announce(k, x, seg_eff + seg_skip, u);
                            if (ok) pad_to(x);
                            if (!ok) break;
                            paged_tile = u.pos.tile;
                            if (u.pos.uid < sc.U) {
                                // the segment's page-table entries, widened to 16-byte pieces, in one bulk copy
                                const int first = u.pos.tile & ~3, last = (u.pos.tile + seg_eff + 3) & ~3;
                                const int* src = pg->page_table + (size_t)pg->seq_slot[u.b] * pg->table_stride + first;
                                mbar_expect_tx(smem_u32(page_bar), (uint32_t)(last - first) * 4u);
                                bulk_load(smem_u32(s_pages), src, (uint32_t)(last - first) * 4u, smem_u32(page_bar));
                                ok = wait_bounded(smem_u32(page_bar), ppar, s_abort, a.status, kStatusPageWaitTimeout);
                                if (!ok) {
                                    page_lost_par = (int)ppar;
                                    break;
                                }
                                ppar ^= 1u;
                                page_base = first;
                                // 16-bit pages: the first pool row of the head's pages; 8-bit pages: its first page
                                const bool whole = pg->step.n_layers > 1;  // per-layer values come per layer
                                paged_row0 = FP8 ? (whole ? pg->page0_8_of[u.layer] : pg->page0_8) + u.slot * pg->n_pages
                                                 : (whole ? pg->step.full_row0[u.layer] : (int)a.full_row0) +
                                                       u.slot * pg->n_pages * 2 * kTile;
                            } else {
                                paged_row0 = -1;
                                const bool whole = pg->step.n_layers > 1;
                                const int c = u.slot;
                                if (FP8) {  // the ring's pages follow one another
                                    ring_next = (whole ? pg->ring0_8_of[u.layer] : pg->ring0_8) +
                                                (pg->seq_slot[u.b] * u.nclass + c) * pg->ring_tiles + u.pos.tile;
                                } else {
                                    krow = (whole ? pg->step.comp_row0[u.layer] : (int)a.comp_row0) +
                                           (pg->seq_slot[u.b] * u.nclass + c) * 2 * a.rows_comp + u.pos.tile * kTile;
                                    vrow = krow + a.rows_comp;
                                }
                            }
                            qsrc = a.q + ((size_t)u.qrow * a.q_heads + (size_t)u.head * G) * D;
                        } else {
                        announce(k, x, seg_left, u);
                        if (ok) pad_to(x);
                        if (!ok) break;
                        // rows the append launch of this step writes: a compressed unit's ring, the
                        // last tile of a full unit (waited for when that tile's turn comes, below).
                        // Everything else is older and may be fetched early.
                        if (early && !synced && (k != (int)blockIdx.x || u.pos.uid >= sc.U)) sync_now();
                        cur_tile = u.pos.tile;
                        newest_tile = u.pos.uid < sc.U ? u.tiles - 1 : -1;
                        if (!MIXED && !STEP && a.new_k) {
                            const int t = a.len_full - 1;  // the token of this step
                            new_row = u.pos.uid < sc.U ? t : (t < a.new_sink ? t : a.new_sink + (t - a.new_sink) % a.new_window);
                            new_tile = new_row / kTile;
                            new_unit_row0 = u.row0;
                            new_vrows = u.vrows;
                            new_src = a.new_k + ((size_t)u.b * (a.q_heads / G) + u.head) * D;
                        }
                        if (MIXED && u.pos.uid >= sc.U) {
                            local_row0 = u.row0;
                            local_next = u.pos.tile;
                        } else {
                            krow = u.row0 + u.pos.tile * kTile;
                            vrow = krow + u.vrows;
                        }
                        qsrc = a.q + ((size_t)u.b * a.q_heads + (size_t)u.head * G) * D;
                        }
                    }
                    // 8-bit pages: the slot holds tiles 2p and 2p + 1 of the unit where the segment has both,
                    // else the one it has, each in its own half of the stage
                    int n_sub = 1, pg0 = 0, pg1 = 0;
                    if (FP8) {
                        n_sub = (paged_tile & 1) ? 1 : min(2, seg_left);
                        if (paged_row0 >= 0) {
                            pg0 = paged_row0 + s_pages[paged_tile - page_base];
                            if (n_sub == 2) pg1 = paged_row0 + s_pages[paged_tile + 1 - page_base];
                        } else {
                            pg0 = ring_next;
                            pg1 = ring_next + 1;
                            ring_next += n_sub;
                        }
                    } else if (PAGED && paged_row0 >= 0) {
                        krow = paged_row0 + s_pages[paged_tile++ - page_base] * (2 * kTile);
                        vrow = krow + kTile;
                    }
                    if (MIXED && local_row0 >= 0) {
                        int row, valid;
                        local_tile(a, local_next++, row, valid);
                        krow = local_row0 + row;
                        vrow = krow + a.rows_full;
                    }
                    if (!PAGED) {
                        // the tile that holds this step's token; a stage whose release depends on query rows
                        // that have not been fetched yet (the ring is full of tiles nobody can consume)
                        if (early && !synced && (cur_tile == newest_tile || (a.dep_wait == 3 && issued >= stages))) sync_now();
                        if (!MIXED && !STEP && cur_tile == new_tile) {
                            // This CTA is the one that reads the tile the step's token belongs to: it writes the
                            // token's K and V rows there itself (a bit-exact copy of the caller's rows), then makes
                            // them visible to the tile copy it issues next.
                            if (early && !synced) sync_now();
                            const uint4* src_k = reinterpret_cast<const uint4*>(new_src);
                            const uint4* src_v = reinterpret_cast<const uint4*>(a.new_v + (new_src - a.new_k));
                            uint4* dst_k = reinterpret_cast<uint4*>(const_cast<__nv_bfloat16*>(a.pool) + (size_t)(new_unit_row0 + new_row) * D);
                            uint4* dst_v = dst_k + (size_t)new_vrows * D / 8;
                            constexpr int N16 = D / 8;  // 16-byte pieces per row
#pragma unroll
                            for (int c0 = 0; c0 < N16; c0 += 8) {
                                uint4 rk[8], rv[8];
#pragma unroll
                                for (int c = 0; c < 8; ++c) {
                                    rk[c] = __ldcg(src_k + c0 + c);
                                    rv[c] = __ldcg(src_v + c0 + c);
                                }
#pragma unroll
                                for (int c = 0; c < 8; ++c) {
                                    dst_k[c0 + c] = rk[c];
                                    dst_v[c0 + c] = rv[c];
                                }
                            }
                            __threadfence();
                            asm volatile("fence.proxy.async;" ::: "memory");
                        }
                        ++cur_tile;
                    }
                    if (trace) cy_seg += clock64() - ts0;
                    ok = wait_traced(smem_u32(empty_bar + s), par ^ 1u, s_abort, a.status, kStatusEmptyWaitTimeout, trace,
                                     &ns_stage);
                    if (!ok) break;
                    const uint32_t fb = smem_u32(full_bar + s);
                    const bool with_q = seg_idx < NG;  // each consumer group reads q at its first tile of the segment
                    const long long tc0 = trace ? clock64() : 0;
                    mbar_expect_tx(fb, (FP8 ? n_sub * (kPairBytes / 2) : kPairBytes) + (with_q ? G * D * 2 : 0));
                    const uint32_t dst = smem_u32(stage_base + (size_t)s * stage_bytes);
                    if (trace && issued == 0) my_trace[37] = global_timer_ns();
                    const long long tc1 = trace ? clock64() : 0;
                    if constexpr (FP8) {
                        // a page in one box of 128 rows of 128 bytes: 64 rows of K codes, then the transposed V
                        // codes, two d per row
                        tma_load_2d(dst + (paged_tile & 1) * (kPairBytes / 2), &extra.map_k, 0, pg0 * 128, fb, stream_policy);
                        if (n_sub == 2) tma_load_2d(dst + kPairBytes / 2, &extra.map_k, 0, pg1 * 128, fb, stream_policy);
                        paged_tile += n_sub;
                    } else if (D == 128) {  // one box per tile, 16 KB contiguous in memory: [2 halves][64 rows][64]
                        tma_load_3d(dst, &tmap, 0, krow, 0, fb, stream_policy);
                        tma_load_3d(dst + S::kTileBytes, &tmap, 0, vrow, 0, fb, stream_policy);
                    } else {         // one contiguous 8 KB box per tile: [64 rows][64]
                        tma_load_2d(dst, &tmap, 0, krow, fb, stream_policy);
                        tma_load_2d(dst + S::kTileBytes, &tmap, 0, vrow, fb, stream_policy);
                    }
                    const long long tc2 = trace ? clock64() : 0;
                    if (with_q) {
                        if (a.dep_wait == 3 && !synced) {  // the query rows are not there yet: fetched at sync_now()
                            late_dst[n_late] = dst + kPairBytes;
                            late_src[n_late] = qsrc;
                            late_bar[n_late++] = fb;
                        } else {
                            bulk_load(dst + kPairBytes, qsrc, G * D * 2, fb);
                        }
                    }
                    if (trace) {
                        const long long tc3 = clock64();
                        cy_expect += tc1 - tc0;
                        cy_tma += tc2 - tc1;
                        cy_q += tc3 - tc2;
                    }
                    krow += kTile;
                    vrow += kTile;
                    ++seg_idx;
                    seg_left -= n_sub;
                    x += n_sub - 1;
                    ++issued;
                    if (++s == stages) {
                        s = 0;
                        par ^= 1u;
                    }
                    if (PAGED && seg_left == 0) x += seg_skip;  // the unit's tiles that do not exist
                }
                if (!ok) break;
                if (early && !synced) sync_now();  // a first item shorter than the ring
                if (PAGED && !asked) mbar_arrive(smem_u32(claim_empty));
                ok = wait_traced(smem_u32(claim_full), cpar, s_abort, a.status, kStatusClaimWaitTimeout, trace, &ns_claim);
                cpar ^= 1u;
                if (ok) k_claim = *claim_slot;
            }
            if (ok) {
                UnitInfo none{};
                announce(-1, 0, 0, none);  // no more work
            }
            if (trace) {
                my_trace[14] = ns_claim;
                my_trace[15] = ns_ring + (ns_stage << 32);
                my_trace[27] = (unsigned long long)(clock64() - t_prod);
                my_trace[32] = (unsigned long long)cy_expect;
                my_trace[33] = (unsigned long long)cy_tma;
                my_trace[34] = (unsigned long long)cy_q;
                my_trace[35] = (unsigned long long)cy_item;
                my_trace[36] = (unsigned long long)cy_seg;
            }
        }
    } else if (warp == S::kWarps + 1) {
        // ------------------------------------------------------------------ claim warp
        if (lane == 0) {
            uint32_t par = 0;
            bool waited = a.dep_wait != 3;  // dep_wait 3: an earlier launch may still be using the claim counter
            for (;;) {
                if (!wait_bounded(smem_u32(claim_empty), par, s_abort, a.status, kStatusClaimWaitTimeout)) break;
                par ^= 1u;
                if (!waited) {
                    grid_dep_wait();
                    waited = true;
                }
                // the counter only ever grows; this launch's claims start at claim_base
                const int k = sc.P + (int)(atomicAdd(a.claim_counter, 1u) - a.claim_base);
                *claim_slot = k;
                mbar_arrive(smem_u32(claim_full));
                if (k >= sc.n_items) break;  // the producer stops asking once it has seen this answer
            }
        } else if (lane == 1 && a.dep_wait == 2) {
            grid_dep_wait();    // the launch before this one has completed ...
            grid_dep_launch();  // ... so the next one, which shares that launch's scratch copy, may start
        }
    } else {
        // ------------------------------------------------------------------ epilogue warps
        constexpr int NE = kEpilogueWarps * 32;
        constexpr int D4 = D / 4;
        const int et = tid - (S::kWarps + 2) * 32;
        const int PF = partial_floats(D, G), PH = partial_head_floats(G);
        // warm the instruction cache with the merge routine while there is nothing else to do: a dry
        // run on unit 0 (its partial records hold whatever the last launch left; nothing is stored).
        // Not in a launch so small that a CTA's stream is a few tiles: there the first segment would
        // wait for the dry run's trip to memory.
        if (sc.n_items > 2 * sc.P) {
            if (et == 0) todo[kMaxTodo - 1] = make_int2(0, 0);
            epilogue_sync();
            if (et < kListStride) {
                int slot = 0, count = 0;
                if (et <= sc.R) unit_partials(sc, 0, et, slot, count);
                // two records per band at most: one batch of loads warms the same instructions as many
                lists[(kMaxTodo - 1) * kListStride + et] = make_int2(slot, count < 2 ? count : 2);
            }
            epilogue_sync();
            merge_units<D, MIXED>(a.partials, a.out, G, sc.R, todo + kMaxTodo - 1, lists + (kMaxTodo - 1) * kListStride,
                                  1, et, NE, true, nullptr, a.alpha, sc.U, a.q_heads, a.out_bf16);
            epilogue_sync();
        }
        if (a.dep_wait == 1 || a.dep_wait == 3) {  // from here on these warps write results, partials and tickets
            grid_dep_wait();
            if (et == 0 && a.dep_wait == 1) grid_dep_launch();
        }
        unsigned long long ns_idle = 0;
        int pend_n = 0;  // partial segments written but without a ticket yet (same value in every epilogue thread)
        const bool tre = trace && et == 0;
        // Draws the tickets of the pending partial segments, all at once: where a segment was its
        // unit's last one the unit goes on the to-do list, merged when the stream has ended (or now,
        // by these warps alone, if the list is full).
        auto flush = [&]() {
            __threadfence();  // this thread's partial stores are visible before any ticket is drawn for them
            epilogue_sync();
            if (*todo_count + pend_n > kMaxTodo) {
                merge_units<D, MIXED>(a.partials, a.out, G, sc.R, todo, lists, *todo_count, et, NE, false, nullptr, a.alpha,
                                      sc.U, a.q_heads, a.out_bf16);
                epilogue_sync();
                if (et == 0) *todo_count = 0;
                epilogue_sync();
            }
            // 16 lanes per pending segment: lane r looks up the unit's partial records in band r (mixed
            // attention: pend holds the pair, i.e. its full unit; lane 15 looks up the local unit's records,
            // which all lie in the last band, and the ticket counts the records of both)
            constexpr int NB = kListStride;
            for (int base = 0; base < pend_n * 16; base += NE) {  // whole warps take part in the shuffles
                const int p = base + et, i = p >> 4, r = p & 15;
                const bool on = p < pend_n * 16;
                int slot = 0, count = 0;
                if (on && r <= sc.R) {
                    if (PAGED) unit_partials(sc, pend[i].x, r, slot, count, paged_unit_tiles(a, pg, pend[i].x));
                    else unit_partials(sc, pend[i].x, r, slot, count);
                }
                if (MIXED && on && r == 15) unit_partials(sc, sc.U + pend[i].x, sc.R, slot, count);
                int total = count;
#pragma unroll
                for (int o = 8; o > 0; o >>= 1) total += __shfl_xor_sync(0xffffffffu, total, o);
                int idx = -1;
                if (on && r == 0 && atomicAdd(&a.tickets[pend[i].x], 1) == total - 1) {
                    a.tickets[pend[i].x] = 0;  // ready for the next launch
                    idx = atomicAdd(todo_count, 1);
                    todo[idx] = pend[i];
                }
                idx = __shfl_sync(0xffffffffu, idx, lane & 16);  // from lane r == 0 of this 16-lane group
                if (idx >= 0 && (r < NB - 1 || r == 15)) lists[idx * NB + (r == 15 ? NB - 1 : r)] = make_int2(slot, count);
            }
            epilogue_sync();
            pend_n = 0;
        };
        for (int seg = 0;; ++seg) {
            const int bi = seg % kMergeBuffers;
            const uint32_t bar = smem_u32(ep_full + bi), bpar = (uint32_t)(seg / kMergeBuffers) & 1u;
            // nothing to merge right now: a good moment to draw tickets (the decision is taken by one
            // thread so that all epilogue threads take the same path)
            if (pend_n > 0) {
                if (et == 0) *ep_flag = mbar_try_wait(bar, bpar) ? 0 : 1;
                epilogue_sync();
                const bool idle = *ep_flag != 0;
                epilogue_sync();
                if (idle || pend_n == kMaxPend) flush();
            }
            const bool got = wait_traced(bar, bpar, s_abort, a.status, kStatusMergeWaitTimeout, tre, &ns_idle);
            if (epilogue_or(!got)) break;
            const uint8_t* buf = buffers + (size_t)bi * buffer_bytes;
            const float* merge = reinterpret_cast<const float*>(buf);
            const float* stat_m = merge + S::merge_floats(G);
            const float* stat_l = stat_m + S::kWarps * kMaxGroup;
            const SegDesc sd = *reinterpret_cast<const SegDesc*>(stat_l + S::kWarps * kMaxGroup);
            if (sd.stop) {
                if (pend_n > 0) flush();
                break;
            }
            float* out_rows = a.out + (size_t)sd.out_row * D;
            float* my_part = a.partials + (size_t)sd.pslot * PF;
            // merge the consumer warps' states; this thread owns a few 4-float pieces of the G x D rows
            for (int e = et; e < G * D4; e += NE) {
                const int g = e / D4, d4 = e - g * D4;
                float M = kNegBig;
#pragma unroll
                for (int w = 0; w < S::kWarps; ++w) M = fmaxf(M, stat_m[w * kMaxGroup + g]);
                float L = 0.f;
                float4 O = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                for (int w = 0; w < S::kWarps; ++w) {
                    const float wt = exp2f(stat_m[w * kMaxGroup + g] - M);
                    const float4 o = *reinterpret_cast<const float4*>(merge + (size_t)(w * G + g) * MS + d4 * 4);
                    L += stat_l[w * kMaxGroup + g] * wt;
                    O.x += o.x * wt;
                    O.y += o.y * wt;
                    O.z += o.z * wt;
                    O.w += o.w * wt;
                }
                if (sd.complete) {
                    const float inv = 1.f / L;
                    if (a.out_bf16)
                        *reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(a.out) + (size_t)sd.out_row * D + e * 4) =
                            make_uint2(pack_bf16(O.x * inv, O.y * inv), pack_bf16(O.z * inv, O.w * inv));
                    else
                        *reinterpret_cast<float4*>(out_rows + e * 4) = make_float4(O.x * inv, O.y * inv, O.z * inv, O.w * inv);
                } else {
                    *reinterpret_cast<float4*>(my_part + PH + e * 4) = O;
                    if (d4 == 0) {
                        my_part[g] = M;
                        my_part[G + g] = L;
                    }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(ep_empty + bi));  // the buffer may be refilled
            if (!sd.complete) {
                // (mixed attention: the pair, named by its full unit)
                if (et == 0) pend[pend_n] = make_int2(MIXED && sd.uid >= sc.U ? sd.uid - sc.U : sd.uid, sd.out_row);
                ++pend_n;
            }
        }
        if (tre) {
            my_trace[7] = global_timer_ns();
            my_trace[11] = ns_idle;
        }
    }
    __syncthreads();
    // ---- the units on this CTA's to-do list: merged by all its warps
    if (trace && tid == 0) my_trace[12] = global_timer_ns();
    if (trace && tid == 0) my_trace[13] = (unsigned long long)*todo_count;
    if (!*s_abort && *todo_count > 0)
        merge_units<D, MIXED>(a.partials, a.out, G, sc.R, todo, lists, *todo_count, tid, S::kThreads, false,
                              trace ? my_trace + 28 : nullptr, a.alpha, sc.U, a.q_heads, a.out_bf16);
    if (warp == S::kWarps && lane == 0) {
        if (*s_abort) {
            // a wait ran out somewhere in this CTA: make sure none of its copies is still in flight
            // when the CTA retires
            for (int j = issued > stages ? issued - stages : 0; j < issued; ++j)
                wait_bounded(smem_u32(full_bar + j % stages), (uint32_t)(j / stages) & 1u, s_abort, a.status,
                             kStatusDrainTimeout, false);
            if (PAGED && page_lost_par >= 0)
                wait_bounded(smem_u32(page_bar), (uint32_t)page_lost_par, s_abort, a.status, kStatusDrainTimeout, false);
        }
    }
    if (trace && tid == 0) my_trace[3] = global_timer_ns();
}

template <int D, int NG, int MODE>
cudaError_t launch_one(const DecodeArgs& a, const CUtensorMap& tmap, int grid, int stages, cudaStream_t stream,
                       bool overlap, const typename ExtraArgs<MODE>::type& extra)
{
    const size_t smem = Smem<D, NG>::bytes(stages, a.group, MODE);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(Smem<D, NG>::kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = overlap ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, decode_kernel<D, NG, MODE>, a, tmap, stages, extra);
}

template <int D, int NG>
cudaError_t prepare_one()
{
    cudaError_t e = cudaFuncSetAttribute(decode_kernel<D, NG, kModePlain>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         kMaxDynamicSmem);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(decode_kernel<D, NG, kModeMixed>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxDynamicSmem);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(decode_kernel<D, NG, kModeStep>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxDynamicSmem);
    if (e != cudaSuccess) return e;
    if (D == 128 && NG == 2) {  // 8-bit pages: head_dim 128, two consumer groups only
        e = cudaFuncSetAttribute(decode_kernel<128, 2, kModePagedFp8>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 kMaxDynamicSmem);
        if (e != cudaSuccess) return e;
    }
    return cudaFuncSetAttribute(decode_kernel<D, NG, kModePaged>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                kMaxDynamicSmem);
}

}  // namespace

size_t decode_smem_bytes(int head_dim, int stages, int group, int groups, int mode)
{
    if (head_dim == 128)
        return groups == 1 ? Smem<128, 1>::bytes(stages, group, mode)
                           : groups == 2 ? Smem<128, 2>::bytes(stages, group, mode) : Smem<128, 3>::bytes(stages, group, mode);
    return groups == 1 ? Smem<64, 1>::bytes(stages, group, mode)
                       : groups == 2 ? Smem<64, 2>::bytes(stages, group, mode) : Smem<64, 3>::bytes(stages, group, mode);
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

template <int D, int NG>
static cudaError_t launch_either(const DecodeArgs& a, const CUtensorMap& tmap, int grid, int stages, cudaStream_t stream,
                                 bool overlap, int mode, const PagedArgs* paged, const StepArgs* step)
{
    if (mode == kModePaged) return launch_one<D, NG, kModePaged>(a, tmap, grid, stages, stream, overlap, *paged);
    if (mode == kModeStep) return launch_one<D, NG, kModeStep>(a, tmap, grid, stages, stream, overlap, *step);
    if (mode == kModeMixed) return launch_one<D, NG, kModeMixed>(a, tmap, grid, stages, stream, overlap, NoPagedArgs{});
    return launch_one<D, NG, kModePlain>(a, tmap, grid, stages, stream, overlap, NoPagedArgs{});
}

cudaError_t launch_decode(const DecodeArgs& a, const CUtensorMap* tmap, int head_dim, int grid,
                          int stages, int groups, cudaStream_t stream, bool overlap, int mode, const PagedArgs* paged,
                          const PagedFp8Args* paged8, const StepArgs* step)
{
    if (mode == kModePaged && !paged) return cudaErrorInvalidValue;
    if (mode == kModeStep && !step) return cudaErrorInvalidValue;
    if (mode == kModePagedFp8) {
        if (!paged8 || head_dim != 128 || groups != 2) return cudaErrorInvalidValue;
        return launch_one<128, 2, kModePagedFp8>(a, *tmap, grid, stages, stream, overlap, *paged8);
    }
    if (head_dim == 128) {
        if (groups == 1) return launch_either<128, 1>(a, *tmap, grid, stages, stream, overlap, mode, paged, step);
        if (groups == 2) return launch_either<128, 2>(a, *tmap, grid, stages, stream, overlap, mode, paged, step);
        return launch_either<128, 3>(a, *tmap, grid, stages, stream, overlap, mode, paged, step);
    }
    if (groups == 1) return launch_either<64, 1>(a, *tmap, grid, stages, stream, overlap, mode, paged, step);
    if (groups == 2) return launch_either<64, 2>(a, *tmap, grid, stages, stream, overlap, mode, paged, step);
    return launch_either<64, 3>(a, *tmap, grid, stages, stream, overlap, mode, paged, step);
}

}  // namespace rlkv
