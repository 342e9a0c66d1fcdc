// Persistent, weight-major routed-MoE decode kernel for sm_100a.
//
// One launch = one decode step of the whole operator (Section 3 of the paper):
//   phase R : router logits, input quantisation (distributed over CTAs), one
//             grid-wide readiness flag, then top-k + routing metadata in every CTA
//   phase U : gate/up projection.  Work = (active expert, 128-wide block of I,
//             128-wide K block of H); the linear list of such k-steps is cut into
//             equal contiguous ranges, one per CTA (split-K across CTAs, partial
//             accumulators exchanged through L2, summed in fixed order)
//   phase D : down projection, same scheme over (active expert, 128-row block of
//             H, 128-wide K block of I); its activation tiles wait on a per-expert
//             readiness flag published by phase U (Section 3.2, readiness-based
//             handoff)
//   reduce  : (token, 128-row block) tasks spread over all CTAs sum the per-slot
//             results in slot order (deterministic, no float atomics)
//
// Warp roles (Section 3.3, warp specialisation): warps 0 and 2 = TMA producers (weight tiles,
// activation tiles), warps 1 and 3 = tcgen05 MMA issuers (even and odd k-steps), warps 4..7 = accumulator/epilogue warps (one TMEM lane
// quadrant each; twice that for 32/64 token columns); all warps share phase R.  Weights are the MMA "A"
// operand (M = 128 weight rows), tokens are the "B" operand with N = 16/32/64 (Eq. 9), K = 32 per instruction,
// four instructions per 128-wide K block; each K block is accumulated in TMEM on its own and scaled by
// (weight block scale x activation group scale) in registers.  Up to 8 tokens the B columns are the step's tokens;
// beyond that, under sparse routing, the columns of a unit are the tokens routed to the unit's expert (compacted:
// gathered activation tile, compact intermediate tile, passes of N tokens for crowded experts).
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp8.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace moe {

constexpr int kBlock = 128;          // weight block edge = activation group = MMA M = K block
constexpr int kRoleWarps = 4;         // warps 0..3: two TMA producers, two MMA issuers
constexpr int kMaxWarps = 12;
constexpr int kEpiWarp0 = 4;         // warps 4..7
constexpr int kEpiGroupThreads = 128; // one accumulator group = 4 warps = the 4 TMEM lane quadrants
constexpr int kMaxStages = 16;
constexpr int kATileBytes = kBlock * kBlock;  // 16 KiB of FP8
constexpr int kMaxTopK = 32;
constexpr int kMaxExperts = 512;
constexpr int kMaxTokens = 128;       // per launch when tokens are compacted per expert; 64 when all tokens are MMA columns
constexpr int kMaxPasses = 8;         // kMaxTokens / 16
constexpr int kMaxUnits = kMaxExperts + kMaxTokens * kMaxTopK / 16;   // virtual experts (expert, pass) of one launch
constexpr int kMaxTmemBufs = 8;      // accumulator buffers in TMEM (one K block each): 8 for N=16, 4 for N=32/64
constexpr int kStampsPerCta = 32;
constexpr int kMaxGrid = 255;         // CTAs the weighted range tables of the compacted variants can hold

// control words at the head of the workspace
// (the two arrival counters are used by alternate launches: a launch counts in one and clears the other)
enum Ctrl { kEpoch = 0, kStatus = 1, kAbort = 2, kRouteCnt = 3, kExitCnt = 5, kRouteCnt2 = 6, kQuantCnt = 8, kDoneCnt = 10, kCtrlWords = 64 };
// device status codes
enum DevStatus { kDevOk = 0, kDevTimeout = 1 };

struct Params {
    int T, H, E, I, K, scoring, renorm;
    float routed_scale;
    int stages;
    int split_slack_kib;            // see range_quantum()
    int split_weight;               // compacted variants: weight of the per-column cost in the range split, in quarters (0: equal k-steps)
    int route_all_tokens;           // up to this many tokens every CTA selects for all of them
    int nr;                         // token rows per expert in hq / hs: the MMA N, or T rounded up to 16 when tokens are compacted per expert
    unsigned long long grid_magic;  // floor(2^40 / grid) + 1: division by the grid size as a multiplication
    unsigned long long timeout_ns;
    const __nv_bfloat16* hidden;
    const __nv_bfloat16* Wr;
    const float* bias;
    const float* W13s;
    const float* W2s;
    __nv_bfloat16* out;
    unsigned* ctrl;
    float* logits;      // [T,E]   (diagnostics: summed router logits, written by CTA 0)
    float* lpart;       // [<=8][T,E] router logits, one slice per K-split part
    int* ids;           // [T,K]
    float* wts;         // [T,K]
    uint8_t* xq;        // [64,H]
    float* xs;          // [T,H/128]
    uint8_t* hq;        // [E,nr,I]
    float* hs;          // [E,I/128,nr]
    unsigned* e_cnt;    // [2][kMaxPasses][E] published I-blocks of an expert's intermediate tile (per launch parity and 16-token pass)
    unsigned* dn_flag;  // [grid] == tag once the CTA has stored every down-projection result of its range
    float* part_up;     // [grid][2N][128]
    float* part_dn;     // [grid][N][128]
    unsigned* pu_flag;  // [grid]
    unsigned* pd_flag;  // [grid]
    float* y;           // [T,K,H]
    unsigned long long* ll;         // [T,E] fused variants: router logits as {launch tag, fp32 bits} words
    unsigned long long* ypl;        // [T,K,I/128,H] fused variants: down-projection partial of every (token, slot, intermediate block), {launch tag, fp32 bits}
    unsigned long long* xsl;        // [clusters][C][2 TC][128] fused variants: partial gate/up sums a cluster exports to the next one, {launch tag, fp32 bits}
    int fsplit;                     // fused variants: cut the group list into equal ranges per cluster (units may be split between two clusters)
    int fC, fnCl;                   // fused variants: CTAs per cluster, clusters in the grid
    int fdyn;                       // fused variants launched in pairs: nonzero = the CTAs work alone when the step has more units than pairs (1: sharing is the expected case, 2: working alone is; +4: long units stay in pairs up to 80 % as many units as CTAs)
    unsigned long long grid_magic1; // ... and then divide by the grid size: floor(2^40 / grid) + 1
    int fkb[9], fhb[9];             // fused variants: rank r of a cluster takes K blocks [fkb[r], fkb[r+1]) and W2 row blocks [fhb[r], fhb[r+1])
    unsigned long long* stamps;     // [grid][32] globaltimer stamps of the phases of the last launch; NULL = none taken
    unsigned long long* stamps_buf; // the same buffer, never NULL (the general variant always records its phases)
    int debug_skip;                 // test hook, bit 0: the fused variants never publish the intermediate tile's readiness (a flag that nothing sets: the waits on it must run out cleanly)
    int stamps_fine;                // fused variants: also stamp inside the routing phase (each stamp costs that phase ~0.1 us)
};

// ---------------------------------------------------------------------------------------------
// PTX wrappers
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
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
__device__ __forceinline__ void fence_barrier_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
// 16-byte asynchronous copy global -> shared (L2 only), and "arrive on the mbarrier once my copies so far have landed"
// (the arrival is one of the barrier's expected count)
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_mbar_arrive(uint32_t bar) {
    asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async;" ::: "memory"); }
// the same for shared memory only: does not wait for this thread's global stores in flight
__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar)
        : "memory");
}
// same, with an L2 eviction-priority hint (weights are read exactly once per step: evict them first, so that the
// small hot data -- flags, partial sums, activation tiles, the kernel's own instructions -- stays in L2)
__device__ __forceinline__ void tma_load_2d_hint(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar, uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3}], [%4], %5;"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar), "l"(policy)
        : "memory");
}
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ void tma_prefetch_desc(const CUtensorMap* map) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}
__device__ __forceinline__ void prefetch_l2(const void* p) { asm volatile("prefetch.global.L2 [%0];" ::"l"(p)); }

__device__ __forceinline__ void tmem_alloc(uint32_t smem_dst, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t addr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(addr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem]^T, FP8 E4M3 operands, fp32 accumulate, M=128, K=32.
__device__ __forceinline__ void umma_f8(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// 32 TMEM lanes x C consecutive 32-bit columns -> C registers per thread (thread = lane, register = column)
template <int C>
__device__ __forceinline__ void tmem_ld(uint32_t taddr, float* v) {
    static_assert(C == 1 || C == 2 || C == 4 || C == 8 || C == 16, "unsupported column count");
    uint32_t r[C];
    if constexpr (C == 1) {
        asm volatile("tcgen05.ld.sync.aligned.32x32b.x1.b32 {%0}, [%1];" : "=r"(r[0]) : "r"(taddr));
    } else if constexpr (C == 2) {
        asm volatile("tcgen05.ld.sync.aligned.32x32b.x2.b32 {%0,%1}, [%2];" : "=r"(r[0]), "=r"(r[1]) : "r"(taddr));
    } else if constexpr (C == 4) {
        asm volatile("tcgen05.ld.sync.aligned.32x32b.x4.b32 {%0,%1,%2,%3}, [%4];"
                     : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(taddr));
    } else if constexpr (C == 8) {
        asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                     : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                     : "r"(taddr));
    } else {
        asm volatile(
            "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
            : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
              "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
            : "r"(taddr));
    }
#pragma unroll
    for (int i = 0; i < C; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ unsigned ld_acquire(const unsigned* p) {
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void red_release_add(unsigned* p, unsigned v) {
    asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void st_release(unsigned* p, unsigned v) {
    asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ unsigned long long gtime() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
__device__ __forceinline__ void epi_bar(int nthreads) { asm volatile("bar.sync 1, %0;" ::"r"(nthreads) : "memory"); }
// barrier over the accumulator threads that also ANDs a predicate, so that give-up decisions are uniform
__device__ __forceinline__ bool epi_all(bool ok, int nthreads) {
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 p, %1, 0;\n\t"
        "bar.red.and.pred q, 1, %2, p;\n\t"
        "selp.u32 %0, 1, 0, q;\n\t}"
        : "=r"(r) : "r"((uint32_t)ok), "r"(nthreads) : "memory");
    return r != 0;
}

#define MOE_STAMP(i) do { if (P.stamps) P.stamps[(size_t)blockIdx.x * kStampsPerCta + (i)] = gtime(); } while (0)
// The general variant takes its sixteen stamps unconditionally (`stamps_buf` always points into the workspace): one
// store per phase and role.  Guarding them was measured 1.3 % SLOWER at 64 tokens (code layout), so they stay.
#define MOE_STAMP_ALWAYS(i) do { P.stamps_buf[(size_t)blockIdx.x * kStampsPerCta + (i)] = gtime(); } while (0)


// K-major, 128-byte swizzled operand tile (rows of 128 bytes, 8-row groups 1024 bytes apart).
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t saddr) {
    return (uint64_t)((saddr >> 4) & 0x3FFF) | (1ull << 16) | (64ull << 32) | (1ull << 46) | (2ull << 61);
}

// ---------------------------------------------------------------------------------------------
// bounded waiting: every spin in this kernel goes through Waiter
// ---------------------------------------------------------------------------------------------
struct Waiter {
    unsigned* ctrl;
    unsigned long long t0, limit;
    bool dead;
    __device__ __forceinline__ void init(unsigned* c, unsigned long long lim) { ctrl = c; t0 = gtime(); limit = lim; dead = false; }
    // called every few hundred polls; returns true when the wait must be given up
    __device__ __noinline__ bool expired(int where) {
        if (*(volatile unsigned*)(ctrl + kAbort) != 0) { dead = true; return true; }
        if (gtime() - t0 > limit) {
            atomicCAS(ctrl + kStatus, 0u, (unsigned)kDevTimeout | ((unsigned)where << 8) | (blockIdx.x << 16));
            atomicExch(ctrl + kAbort, 1u);
            dead = true;
            return true;
        }
        return false;
    }
    __device__ __forceinline__ bool mbar(uint32_t bar, uint32_t parity, int where) {
        if (dead) return false;
        for (uint32_t i = 1;; ++i) {
            if (mbar_try_wait(bar, parity)) return true;
            if ((i & 255u) == 0 && expired(where)) return false;
        }
    }
    __device__ __forceinline__ bool flag(const unsigned* p, unsigned want, int where) {
        if (dead) return false;
        for (uint32_t i = 1;; ++i) {
            if (ld_acquire(p) == want) return true;
            if ((i & 63u) == 0) { if (expired(where)) return false; __nanosleep(64); }
        }
    }
};

// ---------------------------------------------------------------------------------------------
// shared-memory layout
// ---------------------------------------------------------------------------------------------
struct SmemLayout {
    int ring_off, stage_bytes, lo_off, kw_off, pv_off, pv_stride, bar_off, ids_off, w_off, mask_off, act_off, uidx_off, xs_off, hs_off, as_off, red_off, poff_off, pair_off, misc_off, total;
};
__host__ __device__ inline SmemLayout smem_layout(int N, int T, int K, int E, int H, int I, int stages, bool compact, bool weighted) {
    SmemLayout L;
    L.stage_bytes = kATileBytes + N * kBlock;
    L.ring_off = 0;
    int o = stages * L.stage_bytes;
    L.bar_off = o;  o += (3 * kMaxStages + 2 * kMaxTmemBufs + 8) * 8;
    L.misc_off = o; o += 64;
    L.ids_off = o;  o += T * K * 4;
    L.w_off = o;    o += T * K * 4;
    o = (o + 7) & ~7;
    L.mask_off = o; o += E * 16;
    L.act_off = o;  o += (E + 1 + (compact ? (T * K) / N + 1 : 0)) * 4;   // + extra N-token passes of crowded experts
    L.uidx_off = o; o += E * 4;
    o = (o + 15) & ~15;
    L.xs_off = o;   o += ((T + 3) & ~3) * (H / kBlock) * 4;   // input activation scales [H/128][T rounded up to 4]
    L.hs_off = o;   o += N * (I / kBlock) * 4;      // intermediate activation scales of the current expert [I/128][N]  (16-byte aligned rows)
    L.as_off = o;   o += compact ? (N + N * (H / kBlock)) * 4 : 0;   // compacted: tokens of the unit's N columns, their input scales [H/128][N]
    L.red_off = o;  o += kMaxWarps * 64 * 4;        // cross-warp reduction scratch
    L.poff_off = o; o += E * 4;                     // expert -> first entry of its (token, slot) pairs
    L.pair_off = o; o += ((T * K * 2 + 15) & ~15);  // (token | slot << 8) of every routed pair, grouped by expert, tokens ascending
    L.lo_off = o;   o += weighted ? 2 * (kMaxGrid + 1) * 4 : 0;   // weighted ranges: first k-step of every CTA's range, per projection
    L.kw_off = o;   o += weighted ? 2 * 33 * 4 : 0;               // weighted ranges: weight of a k-step by columns in use, per projection
    L.pv_stride = E + (T * K) / N + 2;                           // weighted ranges: weight of the k-steps before every virtual expert, per projection
    L.pv_off = o;   o += weighted ? 2 * L.pv_stride * 4 : 0;
    L.total = o;
    return L;
}

// per-phase split of a linear k-step list into contiguous per-CTA ranges
// (q = 1: equal k-step counts, units may be split between neighbouring CTAs; q = K blocks per unit: whole units only)
// (Sq = number of quanta in the list; the range of CTA c starts at quantum floor(Sq * c / G))
// Integer divisions cost ~100 cycles each on one thread and the range arithmetic sits on the latency-critical path
// between routing and the first weight request, so: division by the grid size is a multiplication by
// magic = floor(2^40 / G) + 1 (exact while a * G < 2^40), small divisions go through a float reciprocal plus fix-up.
__device__ __forceinline__ unsigned div_grid(unsigned a, unsigned long long magic) { return (unsigned)(((unsigned long long)a * magic) >> 40); }
__device__ __forceinline__ int div_small(int a, int d) {          // 0 <= a < 2^22, d > 0
    int q = (int)(__int2float_rz(a) * __frcp_rn(__int2float_rz(d)));
    const int r = a - q * d;
    q += (r >= d) - (r < 0);
    return q;
}
__device__ __forceinline__ int range_lo(int Sq, int c, int q, unsigned long long magic) { return (int)div_grid((unsigned)Sq * (unsigned)c, magic) * q; }

// Ranges of equal weight (compacted variants): `pv[u]` = weight of all k-steps before virtual expert u, pv[U] the total,
// every virtual expert holding n_u k-steps of equal weight.  The range of CTA c starts at the first k-step whose
// preceding weight reaches total * c / G.  Rounded toward zero throughout: the target stays below the total and grows
// with c; every CTA computes the same values, which is all the split needs.
__device__ __forceinline__ unsigned split_target(unsigned total, int c, float rG) {
    return __float2uint_rz(__uint2float_rz(total) * (__int2float_rz(c) * rG));
}
__device__ __forceinline__ int split_point(const unsigned* pv, int a, unsigned target, int n_u, int KB, int q) {   // a = largest u with pv[u] <= target
    const int w = div_small((int)(pv[a + 1] - pv[a]), n_u);
    const int j = min(n_u, div_small((int)(target - pv[a]) + w - 1, w));
    int lo = a * n_u + j;
    if (q != 1) lo = div_small(lo, KB) * KB;                                     // whole units only
    return lo;
}

// Split a projection's units across CTAs (split-K, partial sums exchanged through L2) or keep units whole?
// Whole units cost no exchange but load the busiest CTA with ceil(units/G) units; take them when that surplus,
// in KiB of weight tiles, stays below `slack_kib` (what an exchange costs in streaming time).  Measured: letting
// the down projection of config 2 split at T=8 (surplus 26 KiB) is no faster than whole units.
__device__ __forceinline__ int range_quantum(int units, int KB, int G, int kstep_kib, int slack_kib, unsigned long long magic) {
    const int whole = (int)div_grid((unsigned)(units + G - 1), magic) * KB * kstep_kib;
    const int split = (int)div_grid((unsigned)(units * KB * kstep_kib + G - 1), magic);
    return (whole - split <= slack_kib) ? KB : 1;
}

// position inside the linear k-step list of one projection: k-step -> (K block, row block, active expert)
struct Walk {
    int kb, mb, u, e, KB, MB;
    __device__ __forceinline__ void init(int s, int KB_, int MB_, const int* act) {
        KB = KB_; MB = MB_;
        const int unit = div_small(s, KB);
        kb = s - unit * KB;
        u = div_small(unit, MB);
        mb = unit - u * MB;
        e = act[u];
    }
    __device__ __forceinline__ void next_unit(const int* act) {
        kb = 0;
        if (++mb == MB) { mb = 0; ++u; }
        e = act[u];
    }
    __device__ __forceinline__ void next(const int* act) {
        if (++kb == KB) {
            kb = 0;
            if (++mb == MB) { mb = 0; ++u; }
            e = act[u];
        }
    }
};

// position of the n-th (0-based) set bit of a 64-bit mask that has more than n bits set
__device__ __forceinline__ int nth_set_bit(unsigned long long m, int n) {
    int pos = 0;
#pragma unroll
    for (int w = 32; w; w >>= 1) {
        const int c = __popcll((m >> pos) & ((1ull << w) - 1ull));
        if (n >= c) { pos += w; n -= c; }
    }
    return pos;
}

// Token sets of up to 128 tokens: two 64-bit words per expert (word 0 = tokens 0..63).
struct TokMask { unsigned long long lo, hi; };
__device__ __forceinline__ TokMask load_mask(const unsigned long long* s_mask, int e) { TokMask m; m.lo = s_mask[2 * e]; m.hi = s_mask[2 * e + 1]; return m; }
__device__ __forceinline__ int mask_count(const TokMask& m) { return __popcll(m.lo) + __popcll(m.hi); }
__device__ __forceinline__ int mask_rank(const TokMask& m, int t) {      // members below token t
    return t < 64 ? __popcll(m.lo & ((1ull << t) - 1ull)) : __popcll(m.lo) + __popcll(m.hi & ((1ull << (t - 64)) - 1ull));
}
__device__ __forceinline__ int mask_nth(const TokMask& m, int n) {       // the n-th (0-based) member; needs n < count
    const int c = __popcll(m.lo);
    return n < c ? nth_set_bit(m.lo, n) : 64 + nth_set_bit(m.hi, n - c);
}
__device__ __forceinline__ void mask_add(unsigned long long* s_mask, int e, int t) { atomicOr(&s_mask[2 * e + (t >> 6)], 1ull << (t & 63)); }

// monotone map float -> uint32 (larger float <=> larger integer); +0 and -0 are merged first
__device__ __forceinline__ uint32_t orderable(float f) {
    const uint32_t u = __float_as_uint(f + 0.0f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// Routing (Section 4.1 policies) in two steps.
// (1) route_scores: the whole CTA turns the router logits of a few tokens into selection keys and score values in
//     shared memory: softmax over all experts (key = the logit itself) or sigmoid plus selection bias.
// (2) route_select: one warp per token picks the K largest keys; equal keys go to the lowest expert index; slots
//     are in (key descending, index ascending) order; weights are optionally renormalised over the selected experts.
//     Lane l holds experts l, l+32, ... (NPER of them) in registers.  Selection is K rounds of: warp-wide maximum of
//     the orderable keys (one redux), warp-wide minimum of the indices holding it (one redux), removal of the winner;
//     lane j keeps slot j.  The softmax normaliser is only summed when the weights are not renormalised (it cancels
//     otherwise), with the largest logit -- slot 0 -- as the shift.
// EPT elements per thread and turn, each the sum of up to KP K-split parts: EPT * KP = 16 loads in flight per thread
// (each turn costs an L2 round trip, so few turns matter more than anything else here).
template <int EPT, int KP>
__device__ __forceinline__ void route_scores_t(const Params& P, int t0, int nt, int ksplit, int tid, int nthreads,
                                               uint32_t* s_key, float* s_val, bool write_global) {
    const int E = P.E;
    const bool softmax = (P.scoring == 0);
    for (int p0 = tid; p0 < nt * E; p0 += EPT * nthreads) {
        float part[EPT][KP];                                     // router logit = sum of the K-split parts, fixed order
        float bias[EPT];
#pragma unroll
        for (int j = 0; j < EPT; ++j) {
            const int p = p0 + j * nthreads;
#pragma unroll
            for (int kp = 0; kp < KP; ++kp)
                part[j][kp] = (p < nt * E && kp < ksplit) ? __ldcg(P.lpart + ((size_t)kp * P.T + t0) * E + p) : 0.f;
            bias[j] = (!softmax && P.bias && p < nt * E) ? __ldg(P.bias + (p - div_small(p, E) * E)) : 0.f;
        }
#pragma unroll
        for (int j = 0; j < EPT; ++j) {
            const int p = p0 + j * nthreads;
            if (p < nt * E) {
                float l;                                         // pairwise tree over the parts (absent parts are zeros)
                if constexpr (KP == 2) l = part[j][0] + part[j][1];
                else if constexpr (KP == 4) l = (part[j][0] + part[j][1]) + (part[j][2] + part[j][3]);
                else l = ((part[j][0] + part[j][1]) + (part[j][2] + part[j][3])) + ((part[j][4] + part[j][5]) + (part[j][6] + part[j][7]));
                if (write_global) P.logits[(size_t)t0 * E + p] = l;
                if (softmax) {
                    s_val[p] = l;
                    s_key[p] = orderable(l);
                } else {
                    const float sg = __fdiv_rn(1.0f, 1.0f + expf(-l));
                    s_val[p] = sg;
                    s_key[p] = orderable(sg + bias[j]);
                }
            }
        }
    }
}
__device__ __forceinline__ void route_scores(const Params& P, int t0, int nt, int ksplit, int tid, int nthreads,
                                             uint32_t* s_key, float* s_val, bool write_global) {
    if (ksplit <= 2) route_scores_t<8, 2>(P, t0, nt, ksplit, tid, nthreads, s_key, s_val, write_global);
    else if (ksplit <= 4) route_scores_t<4, 4>(P, t0, nt, ksplit, tid, nthreads, s_key, s_val, write_global);
    else route_scores_t<2, 8>(P, t0, nt, ksplit, tid, nthreads, s_key, s_val, write_global);
}

// Second half of the routing of one token (one warp; lane j < K holds the expert of slot j in `my_id`), in two steps so
// that a caller can put a barrier between them: route_vals() reads what it needs from the score table (the selected
// scores; the softmax normaliser over all experts when the weights are not renormalised), route_weights() turns that
// into the routing weights -- softmax or plain sigmoid score, optionally renormalised over the selected experts, times
// the routed scaling factor (Section 4.1) -- and writes the token's ids and weights.
__device__ __forceinline__ float route_vals(const Params& P, int lane, int my_id, const float* s_val, float& total) {
    const int E = P.E, K = P.K;
    const float v = (lane < K) ? s_val[my_id] : 0.f;
    total = 1.0f;
    if (P.scoring == 0 && !P.renorm) {
        const float mx = __shfl_sync(0xffffffffu, v, 0);        // slot 0 holds the largest logit
        total = 0.f;
        for (int e = lane; e < E; e += 32) total += expf(s_val[e] - mx);
#pragma unroll
        for (int o = 16; o; o >>= 1) total += __shfl_xor_sync(0xffffffffu, total, o);
    }
    return v;
}
__device__ __forceinline__ void route_weights(const Params& P, int t, int lane, int my_id, float v, float total,
                                              int* s_ids, float* s_w, bool write_global) {
    const int K = P.K;
    if (P.scoring == 0) {
        const float mx = __shfl_sync(0xffffffffu, v, 0);
        v = (lane < K) ? expf(v - mx) : 0.f;
    }
    float vsum = v;
#pragma unroll
    for (int o = 16; o; o >>= 1) vsum += __shfl_xor_sync(0xffffffffu, vsum, o);
    if (lane < K) {
        const float w = __fdiv_rn(v, P.renorm ? vsum : total) * P.routed_scale;
        s_ids[t * K + lane] = my_id;
        s_w[t * K + lane] = w;
        if (write_global) { P.ids[t * K + lane] = my_id; P.wts[t * K + lane] = w; }
    }
}
__device__ __forceinline__ void route_finish(const Params& P, int t, int lane, int my_id, const float* s_val,
                                             int* s_ids, float* s_w, unsigned long long* s_mask, bool write_global, bool build_mask) {
    float total;
    const float v = route_vals(P, lane, my_id, s_val, total);
    route_weights(P, t, lane, my_id, v, total, s_ids, s_w, write_global);
    if (build_mask && lane < P.K) mask_add(s_mask, my_id, t);
}

template <int NPER>
__device__ __forceinline__ void route_select(const Params& P, int t, int lane, const uint32_t* s_key, const float* s_val,
                                             int* s_ids, float* s_w, unsigned long long* s_mask, bool write_global, bool build_mask) {
    const int E = P.E, K = P.K;
    uint32_t key[NPER];
#pragma unroll
    for (int i = 0; i < NPER; ++i) key[i] = (i * 32 + lane < E) ? s_key[i * 32 + lane] : 0u;    // 0 is below every real key
    int my_id = 0;
#pragma unroll 1
    for (int j = 0; j < K; ++j) {                              // (a serial chain: unrolling buys nothing, and code fetched once per launch is dear)
        uint32_t m = key[0];
#pragma unroll
        for (int i = 1; i < NPER; ++i) m = max(m, key[i]);
        const uint32_t wm = __reduce_max_sync(0xffffffffu, m);
        int cand = 0x7fffffff;
#pragma unroll
        for (int i = NPER - 1; i >= 0; --i) cand = (key[i] == wm) ? i * 32 : cand;
        const int we = __reduce_min_sync(0xffffffffu, cand == 0x7fffffff ? cand : cand + lane);
        const int mine = we - lane;                            // i * 32 if this lane holds the winner
#pragma unroll
        for (int i = 0; i < NPER; ++i) key[i] = (mine == i * 32) ? 0u : key[i];
        if (lane == j) my_id = we;
    }
    route_finish(P, t, lane, my_id, s_val, s_ids, s_w, s_mask, write_global, build_mask);
}

// The selection alone: slot j's expert ends up in lane j (returned), the ids and the token masks are written; the
// routing weights follow later through route_finish() (only the final reduction needs them).
template <int NPER>
__device__ __forceinline__ int route_pick(const Params& P, int t, int lane, const uint32_t* s_key, int* s_ids, unsigned long long* s_mask) {
    const int E = P.E, K = P.K;
    uint32_t key[NPER];
#pragma unroll
    for (int i = 0; i < NPER; ++i) key[i] = (i * 32 + lane < E) ? s_key[i * 32 + lane] : 0u;    // 0 is below every real key
    int my_id = 0;
#pragma unroll 1
    for (int j = 0; j < K; ++j) {
        uint32_t m = key[0];
#pragma unroll
        for (int i = 1; i < NPER; ++i) m = max(m, key[i]);
        const uint32_t wm = __reduce_max_sync(0xffffffffu, m);
        int cand = 0x7fffffff;
#pragma unroll
        for (int i = NPER - 1; i >= 0; --i) cand = (key[i] == wm) ? i * 32 : cand;
        const int we = __reduce_min_sync(0xffffffffu, cand == 0x7fffffff ? cand : cand + lane);
        const int mine = we - lane;                            // i * 32 if this lane holds the winner
#pragma unroll
        for (int i = 0; i < NPER; ++i) key[i] = (mine == i * 32) ? 0u : key[i];
        if (lane == j) my_id = we;
    }
    if (lane < K) { s_ids[t * K + lane] = my_id; mask_add(s_mask, my_id, t); }
    return my_id;
}

// quantise 4 floats with scale s into 4 E4M3 bytes (memory order x0..x3)
__device__ __forceinline__ uint32_t quant4(float x0, float x1, float x2, float x3, float s) {
    float2 a = make_float2(__fdiv_rn(x0, s), __fdiv_rn(x1, s));
    float2 b = make_float2(__fdiv_rn(x2, s), __fdiv_rn(x3, s));
    uint32_t lo = __nv_cvt_float2_to_fp8x2(a, __NV_SATFINITE, __NV_E4M3);
    uint32_t hi = __nv_cvt_float2_to_fp8x2(b, __NV_SATFINITE, __NV_E4M3);
    return lo | (hi << 16);
}

// ---------------------------------------------------------------------------------------------
// the kernel
// N  = MMA N (token tile, 16/32/64); TC = token columns the accumulator warps actually read (power of two >= T).
// WS = ranges of equal weight instead of equal k-step counts (compacted variants only; a variant of its own because
//      even unexecuted code in the accumulator loops costs the small-batch cases a microsecond or two).
// ---------------------------------------------------------------------------------------------
// Accumulator warps: one group of 4 warps for TC <= 16, two groups (each half of the token columns) for TC >= 32.
template <int N, int TC, bool WS = false>
__global__ void __launch_bounds__(128 + 128 * (TC >= 32 ? 2 : 1), 1)
moe_decode_kernel(const __grid_constant__ CUtensorMap tmW13, const __grid_constant__ CUtensorMap tmW2,
                  const __grid_constant__ CUtensorMap tmXq, const __grid_constant__ CUtensorMap tmHq,
                  const __grid_constant__ Params P) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);

    // Tokens compacted per expert (N = TC = 16 or 32, used for more than 8 tokens): the N MMA columns of a unit are
    // the tokens routed to its expert, not all tokens of the step, so the accumulator work follows the routed pairs;
    // an expert with more than N tokens is walked in passes of N (its weights stream once per pass).
    constexpr bool kCompact = (TC >= 16 && TC == N && N <= 32);
    constexpr int kEpiGroups = (TC >= 32) ? 2 : 1;
    constexpr int kEpiThreads = kEpiGroupThreads * kEpiGroups;
    constexpr int kThreads = 128 + kEpiThreads, kWarps = kThreads / 32;
    constexpr int TCG = TC / kEpiGroups;                         // token columns per accumulator group
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int cta = blockIdx.x, G = gridDim.x;
    const int T = P.T, H = P.H, E = P.E, I = P.I, K = P.K;
    const int KBu = H / kBlock, IB = I / kBlock, HB = H / kBlock, KBd = IB;
    const int S = P.stages;
    const SmemLayout L = smem_layout(N, T, K, E, H, I, S, kCompact, WS);
    const int TS = (T + 3) & ~3;                              // token stride of the transposed input scales

    uint64_t* bars = (uint64_t*)(smem + L.bar_off);
    const uint32_t bar_full = smem_u32(bars), bar_empty = smem_u32(bars + kMaxStages);
    constexpr int kTmemBufs = (N <= 32) ? 8 : 4;                 // 8 x 32 = 256, 8 x 64 = 512, 4 x 128 = 512 columns
    constexpr int kBufShift = (N <= 32) ? 3 : 2;
    const uint32_t bar_fullb = smem_u32(bars + 2 * kMaxStages);  // activation tile landed (second producer)
    const uint32_t bar_tfull = smem_u32(bars + 3 * kMaxStages), bar_tempty = smem_u32(bars + 3 * kMaxStages + kMaxTmemBufs);
    const uint32_t bar_drain = smem_u32(bars + 3 * kMaxStages + 2 * kMaxTmemBufs);
    uint32_t* misc = (uint32_t*)(smem + L.misc_off);  // [0] tmem base, [1] U, [2] routing published, [3] give-up flag of the accumulator warps, [4],[5] k-steps issued by the two MMA issuers
    int* s_ids = (int*)(smem + L.ids_off);
    float* s_w = (float*)(smem + L.w_off);
    unsigned long long* s_mask = (unsigned long long*)(smem + L.mask_off);
    int* s_act = (int*)(smem + L.act_off);
    int* s_uidx = (int*)(smem + L.uidx_off);               // expert -> position in the active list
    float* s_xs = (float*)(smem + L.xs_off);
    float* s_hs = (float*)(smem + L.hs_off);
    float* s_red = (float*)(smem + L.red_off);
    int* s_utok = (int*)(smem + L.as_off);                  // compacted only
    int* s_poff = (int*)(smem + L.poff_off);
    unsigned short* s_pair = (unsigned short*)(smem + L.pair_off);
    float* s_as = (float*)(smem + L.as_off) + N;

    // Programmatic dependent launch: let the next launch in the stream start placing its CTAs as ours retire, and
    // do not touch any global memory before the previous launch has completed and flushed (both are no-ops when the
    // launch was not made with the programmatic-serialization attribute).
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    // Set-up that touches only this CTA's shared and tensor memory runs before the wait on the previous launch.
    constexpr uint32_t kTmemCols = kTmemBufs * 2 * N;            // buffers x (gate N + up N) columns: 256/512/512
    if (warp == 0 && lane == 0) {
        tma_prefetch_desc(&tmW13); tma_prefetch_desc(&tmW2); tma_prefetch_desc(&tmXq); tma_prefetch_desc(&tmHq);
        for (int s = 0; s < S; ++s) { mbar_init(bar_full + 8 * s, 1); mbar_init(bar_fullb + 8 * s, kCompact ? 32 : 1); mbar_init(bar_empty + 8 * s, 1); }
        for (int b = 0; b < kTmemBufs; ++b) { mbar_init(bar_tfull + 8 * b, 1); mbar_init(bar_tempty + 8 * b, 4 * kEpiGroups); }
        mbar_init(bar_drain, 1);
        mbar_init(bar_drain + 16, 1);
        misc[3] = 0u; misc[4] = 0u; misc[5] = 0u; misc[6] = 0u; misc[7] = 0u;
        fence_barrier_init();
    }
    if (warp == 1) { tmem_alloc(smem_u32(misc), kTmemCols); tmem_relinquish(); }
#pragma unroll 1
    for (int e = tid; e < 2 * E; e += kThreads) s_mask[e] = 0ull;
    int ksplit = 1;                                              // parts of H per router tile: enough to occupy the grid
    {
        const int items = ((E + 15) / 16) * ((T + 7) / 8);
        while (ksplit < 8 && items * ksplit * 2 <= G && H % (32 * ksplit) == 0 && H / (2 * ksplit) >= 128) ksplit *= 2;
        // Router weights of this CTA's first tile: ask L2 for them now (a prefetch reads nothing into the SM, and L2
        // is the point of coherence, so this is safe ahead of the wait whatever the previous launch wrote).
        const int nTB = (T + 7) / 8;
        if (cta < ((E + 15) / 16) * nTB * ksplit) {
            const int item = cta / ksplit, kp = cta - item * ksplit, eb = item / nTB;
            const int kpart_len = H / ksplit;
            const int kper = (kpart_len / 16 + kWarps - 1) / kWarps * 16;
            const int k_lo = kp * kpart_len + warp * kper, k_hi = min((kp + 1) * kpart_len, k_lo + kper);
            const int lines = (k_hi - k_lo + 63) / 64;                        // 128-byte lines per row
#pragma unroll 1
            for (int idx = lane; idx < 16 * lines; idx += 32) {
                const int r = eb * 16 + (idx & 15);
                if (r < E) prefetch_l2(P.Wr + (size_t)r * H + k_lo + (idx >> 4) * 64);
            }
        }
    }
    asm volatile("griddepcontrol.wait;" ::: "memory");
    Waiter wt;
    wt.init(P.ctrl, P.timeout_ns);
    const unsigned tag = ld_acquire(P.ctrl + kEpoch) + 1u;
    if (tid == 0) MOE_STAMP_ALWAYS(0);
    const unsigned par = tag & 1u;
    unsigned* e_cnt = P.e_cnt + par * kMaxPasses * E;       // counters of this launch: [pass][expert]
#pragma unroll 1
    for (int e = cta * kThreads + tid; e < kMaxPasses * E; e += G * kThreads) P.e_cnt[(par ^ 1u) * kMaxPasses * E + e] = 0u;
    if (cta == 0 && tid == 0) {
        P.ctrl[kRouteCnt + (par ^ 1u)] = 0u; P.ctrl[kRouteCnt2 + (par ^ 1u)] = 0u;
        P.ctrl[kQuantCnt + (par ^ 1u)] = 0u; P.ctrl[kDoneCnt + (par ^ 1u)] = 0u;      // (counters of the fused variants, which may share the workspace)
    }
    if (P.bias && tid * 32 < E) prefetch_l2(P.bias + tid * 32);

    // ------------------------------------------------------------------ phase R: quantise + logits
    {
        // input quantisation: one warp per (token, 128-column group)  (Section 4.1)
        const int groups = T * KBu;
#pragma unroll 1
        for (int p = (G - 1 - cta) * kWarps + warp; p < groups; p += G * kWarps) {   // from the last CTA down: the first ones have router tiles
            const int t = p / KBu, g = p % KBu;
            const uint2 raw = *reinterpret_cast<const uint2*>(P.hidden + (size_t)t * H + g * kBlock + lane * 4);
            const float x0 = __uint_as_float(raw.x << 16), x1 = __uint_as_float(raw.x & 0xFFFF0000u);
            const float x2 = __uint_as_float(raw.y << 16), x3 = __uint_as_float(raw.y & 0xFFFF0000u);
            float amax = fmaxf(fmaxf(fabsf(x0), fabsf(x1)), fmaxf(fabsf(x2), fabsf(x3)));
#pragma unroll
            for (int o = 16; o; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
            const float s = __fdiv_rn(fmaxf(amax, 1e-10f), 448.0f);
            *reinterpret_cast<uint32_t*>(P.xq + (size_t)t * H + g * kBlock + lane * 4) = quant4(x0, x1, x2, x3, s);
            if (lane == 0) P.xs[p] = s;
        }
        if (tid == 0) MOE_STAMP_ALWAYS(1);
        // Router logits (Section 3.3): a (16 experts x 8 tokens) tile and one of `ksplit` parts of H per CTA turn; the
        // CTA's warps split that part of H, each accumulates with warp-level bf16 MMAs (m16n8k16, fp32 accumulate)
        // straight from global memory, the warps' partial tiles are summed in warp order, and the K-split parts are
        // summed in part order by whoever reads the logits (deterministic).  The router is ~0.01 % of the step's
        // flops: this is about latency and about spreading the reads of Wr over all SMs, not about the tensor pipe.
        {
            float* tile = reinterpret_cast<float*>(smem);               // [kWarps][32 lanes][4] partial tiles
            const int nEB = (E + 15) / 16, nTB = (T + 7) / 8;
            const int g = lane >> 2, tq = lane & 3;
            const int kpart_len = H / ksplit;
            const int kper = (kpart_len / 16 + kWarps - 1) / kWarps * 16;   // K range of one warp (multiple of 16)
#pragma unroll 1
            for (int wi = cta; wi < nEB * nTB * ksplit; wi += G) {
                const int item = wi / ksplit, kp = wi - item * ksplit;
                const int eb = item / nTB, tb = item - eb * nTB;
                const int r0 = eb * 16 + g, r1 = r0 + 8, tok = tb * 8 + g;
                const uint32_t* a0p = reinterpret_cast<const uint32_t*>(P.Wr + (size_t)(r0 < E ? r0 : 0) * H);
                const uint32_t* a1p = reinterpret_cast<const uint32_t*>(P.Wr + (size_t)(r1 < E ? r1 : 0) * H);
                const uint32_t* bp = reinterpret_cast<const uint32_t*>(P.hidden + (size_t)(tok < T ? tok : 0) * H);
                float c[4] = {0.f, 0.f, 0.f, 0.f};
                const int k_lo = kp * kpart_len + warp * kper, k_hi = min((kp + 1) * kpart_len, k_lo + kper);
#pragma unroll 8
                for (int k = k_lo; k < k_hi; k += 16) {
                    const int o = (k >> 1) + tq;                          // 32-bit word holding elements k+2tq, k+2tq+1
                    const uint32_t a0 = __ldg(a0p + o), a1 = __ldg(a1p + o), a2 = __ldg(a0p + o + 4), a3 = __ldg(a1p + o + 4);
                    const uint32_t b0 = __ldg(bp + o), b1 = __ldg(bp + o + 4);
                    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
                }
                *reinterpret_cast<float4*>(tile + (warp * 32 + lane) * 4) = make_float4(c[0], c[1], c[2], c[3]);
                __syncthreads();
                if (tid < 128) {
                    float v = 0.f;
                    for (int w = 0; w < kWarps; ++w) v += tile[w * 128 + tid];
                    const int ln = tid >> 2, i = tid & 3;
                    const int row = eb * 16 + (ln >> 2) + (i >= 2 ? 8 : 0), col = tb * 8 + 2 * (ln & 3) + (i & 1);
                    if (row < E && col < T) P.lpart[((size_t)kp * T + col) * E + row] = v;
                }
                __syncthreads();
            }
        }
    }
    if (tid == 0) MOE_STAMP_ALWAYS(2);
    // publish: generic writes of xq must be visible to the async proxy (TMA) of every CTA
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = misc[0];
    static_assert(!WS || (TC >= 16 && TC == N && N <= 32), "weighted ranges exist for the compacted variants only");
    constexpr bool wsplit = WS;   // ranges of equal weight instead of equal k-step counts (see below)
    if constexpr (kCompact) {
        // weight of one k-step of a unit with c columns in use, c = 0..N, per projection (computed while thread 0 waits)
        if (wsplit && tid >= 32 && tid <= 32 + N) {
            const int c = tid - 32;
            unsigned* s_kw = (unsigned*)(smem + L.kw_off);
            s_kw[c] = 64u + (unsigned)((P.split_weight * (c / 4 + min(64, div_small(4 * c, KBu)))) >> 2);
            s_kw[33 + c] = 64u + (unsigned)((P.split_weight * (c + min(64, div_small(8 * c, KBd)))) >> 2);
        }
    }
    if (tid == 0) {
        MOE_STAMP_ALWAYS(3);
        red_release_add(P.ctrl + kRouteCnt + par, 1u);      // all CTAs' logits and xq published once this reaches G
        const bool ok = wt.flag(P.ctrl + kRouteCnt + par, (unsigned)G, 1);
        misc[2] = ok ? 1u : 0u;
        MOE_STAMP_ALWAYS(4);
    }
    __syncthreads();
    bool alive = (misc[2] != 0u);

    // ------------------------------------------------------------------ top-k + routing metadata (every CTA)
    if (alive) {
        // input scales, transposed to [K block][token]: the first load is issued here and consumed after the routing loads
        const float xs0 = (tid < T * KBu) ? __ldcg(P.xs + tid) : 0.f;
        // few tokens: every CTA selects for all of them (no second grid-wide wait); many tokens: CTAs share the
        // tokens (one each, up to the grid size), publish ids and weights, and everybody reads all of them after a second
        // arrival counter (two more L2 round trips).  The idle weight ring holds the keys and score values.
        constexpr bool kAlwaysAll = (TC <= 8);             // the token-column variants serve at most 8 tokens: no shared routing code in them
        // (keys and score values of all tokens go into the idle weight ring: they have to fit what the stage count leaves)
        const bool route_all = kAlwaysAll || ((T <= P.route_all_tokens) && (T * E <= 8192) && (2 * T * E * 4 <= S * L.stage_bytes));
        const int tpc = (T + G - 1) / G;                   // tokens per selecting CTA when the grid shares them (1 up to G tokens)
        const int n_route_ctas = (T + tpc - 1) / tpc;
        const int rt0 = route_all ? 0 : min(T, cta * tpc), rnt = route_all ? T : min(T - rt0, tpc);
        uint32_t* s_key = reinterpret_cast<uint32_t*>(smem);
        float* s_val = reinterpret_cast<float*>(smem) + rnt * E;
        const bool wg = route_all ? (cta == 0) : true;
        route_scores(P, rt0, rnt, ksplit, tid, kThreads, s_key, s_val, wg);
        if (tid < T * KBu) { const int tt = div_small(tid, KBu); s_xs[(tid - tt * KBu) * TS + tt] = xs0; }
        for (int i0 = tid + kThreads; i0 < T * KBu; i0 += 8 * kThreads) {          // the rest, eight loads in flight per thread
            float v[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) v[j] = (i0 + j * kThreads < T * KBu) ? __ldcg(P.xs + i0 + j * kThreads) : 0.f;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int i = i0 + j * kThreads;
                if (i < T * KBu) { const int tt = div_small(i, KBu); s_xs[(i - tt * KBu) * TS + tt] = v[j]; }
            }
        }
        __syncthreads();
        if (tid == 0) MOE_STAMP_ALWAYS(5);
#pragma unroll 1
        for (int tl = warp; tl < rnt; tl += kWarps) {
            const int t = rt0 + tl;
            if (E <= 128) route_select<4>(P, t, lane, s_key + tl * E, s_val + tl * E, s_ids, s_w, s_mask, wg, route_all);
            else if (E <= 256) route_select<8>(P, t, lane, s_key + tl * E, s_val + tl * E, s_ids, s_w, s_mask, wg, route_all);
            else route_select<16>(P, t, lane, s_key + tl * E, s_val + tl * E, s_ids, s_w, s_mask, wg, route_all);
        }
        __syncthreads();
        if (!kAlwaysAll && !route_all) {
            if (tid == 0) {
                if (cta < n_route_ctas) red_release_add(P.ctrl + kRouteCnt2 + par, 1u);
                const bool ok = wt.flag(P.ctrl + kRouteCnt2 + par, (unsigned)n_route_ctas, 12);
                misc[2] = ok ? 1u : 0u;
            }
            __syncthreads();
            alive = (misc[2] != 0u);
            if (alive) {
                for (int i0 = tid; i0 < T * K; i0 += 4 * kThreads) {                 // eight loads in flight per thread
                    int id[4];
                    float wv[4];
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const int i = i0 + j * kThreads;
                        id[j] = (i < T * K) ? __ldcg(P.ids + i) : 0;
                        wv[j] = (i < T * K) ? __ldcg(P.wts + i) : 0.f;
                    }
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const int i = i0 + j * kThreads;
                        if (i < T * K) { s_ids[i] = id[j]; s_w[i] = wv[j]; mask_add(s_mask, id[j], div_small(i, K)); }
                    }
                }
            }
            __syncthreads();
        }
        if (tid == 0) MOE_STAMP_ALWAYS(6);
        if constexpr (kCompact && !WS) {
            // active list in ascending expert order, entry = expert | pass << 16 (passes of N tokens): every warp takes
            // 32-expert chunks; the chunks' totals meet in shared memory (the idle weight ring)
            int* s_tot = reinterpret_cast<int*>(smem);
            const int nch = (E + 31) / 32;
            for (int c = warp; c < nch; c += kWarps) {
                const int e = c * 32 + lane;
                const int np = (e < E) ? (mask_count(load_mask(s_mask, e)) + N - 1) / N : 0;
                const int tot = __reduce_add_sync(0xffffffffu, np);
                if (lane == 0) s_tot[c] = tot;
            }
            __syncthreads();
            for (int c = warp; c < nch; c += kWarps) {
                const int e = c * 32 + lane;
                const int np = (e < E) ? (mask_count(load_mask(s_mask, e)) + N - 1) / N : 0;
                int incl = np;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) { const int v = __shfl_up_sync(0xffffffffu, incl, o); if (lane >= o) incl += v; }
                const int base = __reduce_add_sync(0xffffffffu, (lane < c) ? s_tot[lane] : 0);   // nch <= 16 chunks
                const int u0 = base + incl - np;
                for (int ps = 0; ps < np; ++ps) s_act[u0 + ps] = e | (ps << 16);
                if (np) s_uidx[e] = u0;
                if (c == nch - 1 && lane == 31) { misc[1] = (uint32_t)(base + incl); s_act[base + incl] = 0; }
            }
        } else if constexpr (kCompact) {
            // active list in ascending expert order, entry = expert | pass << 16 (passes of N tokens): every warp takes
            // 32-expert chunks; the chunks' totals meet in shared memory (the idle weight ring).  The same scan carries
            // the weights of the range split (see below): s_pv[ph][u] = weight of all k-steps before virtual expert u.
            int* s_tot = reinterpret_cast<int*>(smem);                          // [3][32] chunk totals: passes, up weight, down weight
            unsigned* s_pv = (unsigned*)(smem + L.pv_off);                      // [2][pv_stride]
            const int PVS = L.pv_stride;
            const int nch = (E + 31) / 32;
            const unsigned n_up_u = (unsigned)(IB * KBu), n_dn_u = (unsigned)(HB * KBd);   // k-steps of one virtual expert
            const unsigned* s_kw = (const unsigned*)(smem + L.kw_off);
            const unsigned wfu = wsplit ? s_kw[N] * n_up_u : 0u, wfd = wsplit ? s_kw[33 + N] * n_dn_u : 0u;   // a full pass
            constexpr int kIters = (kMaxExperts / 32 + kWarps - 1) / kWarps;    // chunks per warp (unrolled: the arrays stay in registers)
            int np_l[kIters];
            unsigned wu_l[kIters], wd_l[kIters];
#pragma unroll
            for (int it = 0; it < kIters; ++it) {
                const int c = warp + it * kWarps;
                if (c >= nch) break;
                const int e = c * 32 + lane;
                const int m = (e < E) ? mask_count(load_mask(s_mask, e)) : 0;
                const int full = m / N, rem = m - full * N;
                const unsigned wru = (wsplit && rem) ? s_kw[rem] * n_up_u : 0u, wrd = (wsplit && rem) ? s_kw[33 + rem] * n_dn_u : 0u;
                np_l[it] = full + (rem != 0); wu_l[it] = (unsigned)full * wfu + wru; wd_l[it] = (unsigned)full * wfd + wrd;
                const int tot = __reduce_add_sync(0xffffffffu, np_l[it]);
                if (lane == 0) s_tot[c] = tot;
                if (wsplit) {
                    const unsigned tu = __reduce_add_sync(0xffffffffu, wu_l[it]), td = __reduce_add_sync(0xffffffffu, wd_l[it]);
                    if (lane == 0) { s_tot[32 + c] = (int)tu; s_tot[64 + c] = (int)td; }
                }
            }
            __syncthreads();
#pragma unroll
            for (int it = 0; it < kIters; ++it) {
                const int c = warp + it * kWarps;
                if (c >= nch) break;
                const int e = c * 32 + lane;
                const int np = np_l[it];
                int incl = np;
                unsigned iu = wu_l[it], id = wd_l[it];
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) { const int v = __shfl_up_sync(0xffffffffu, incl, o); if (lane >= o) incl += v; }
                const int base = __reduce_add_sync(0xffffffffu, (lane < c) ? s_tot[lane] : 0);   // nch <= 16 chunks
                const int u0 = base + incl - np;
                for (int ps = 0; ps < np; ++ps) s_act[u0 + ps] = e | (ps << 16);
                if (np) s_uidx[e] = u0;
                if (c == nch - 1 && lane == 31) { misc[1] = (uint32_t)(base + incl); s_act[base + incl] = 0; }
                if (wsplit) {
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) {
                        const unsigned vu = __shfl_up_sync(0xffffffffu, iu, o), vd = __shfl_up_sync(0xffffffffu, id, o);
                        if (lane >= o) { iu += vu; id += vd; }
                    }
                    const unsigned bu = __reduce_add_sync(0xffffffffu, (lane < c) ? (unsigned)s_tot[32 + lane] : 0u);
                    const unsigned bd = __reduce_add_sync(0xffffffffu, (lane < c) ? (unsigned)s_tot[64 + lane] : 0u);
                    const unsigned pu0 = bu + iu - wu_l[it], pd0 = bd + id - wd_l[it];
                    for (int ps = 0; ps < np; ++ps) { s_pv[u0 + ps] = pu0 + (unsigned)ps * wfu; s_pv[PVS + u0 + ps] = pd0 + (unsigned)ps * wfd; }
                    if (c == nch - 1 && lane == 31) { s_pv[base + incl] = bu + iu; s_pv[PVS + base + incl] = bd + id; }
                }
            }
        } else if (warp == 0) {                            // active list in ascending expert order
            int base = 0;
#pragma unroll 1
            for (int e0 = 0; e0 < E; e0 += 32) {
                const int e = e0 + lane;
                const bool on = (e < E) && (s_mask[2 * e] != 0ull);
                const unsigned b = __ballot_sync(0xffffffffu, on);
                if (on) { const int u = base + __popc(b & ((1u << lane) - 1u)); s_act[u] = e; s_uidx[e] = u; }
                base += __popc(b);
            }
            if (lane == 0) { misc[1] = (uint32_t)base; s_act[base] = 0; }
        }
        __syncthreads();
    }
    const int U = alive ? (int)misc[1] : 0;
    if (tid == 0) MOE_STAMP_ALWAYS(7);
    const int S_up = U * IB * KBu, S_dn = U * HB * KBd;     // k-steps of the two projections (host checks the range)
    const unsigned long long gm = P.grid_magic;
    const int q_up = range_quantum(U * IB, KBu, G, 32, P.split_slack_kib, gm), q_dn = range_quantum(U * HB, KBd, G, 16, P.split_slack_kib, gm);
    const int Sq_up = (q_up == 1) ? S_up : U * IB, Sq_dn = (q_dn == 1) ? S_dn : U * HB;      // quanta per list
    // Range of CTA c in projection ph (0 up, 1 down).  Token-column variants: equal numbers of k-steps (closed form).
    // Compacted variants: the accumulator warps pay per column in use, so a k-step of an expert with many tokens is
    // dearer than one of an expert with few; there the list is cut into ranges of equal WEIGHT, a k-step of a unit
    // with `cnt` columns in use weighing 64 + cnt/4 + 4 cnt/(K blocks) going up and 64 + cnt + 8 cnt/(K blocks) going
    // down (fitted to the measured per-CTA phase times; the second term is the per-unit epilogue spread over the
    // unit's k-steps).  Every CTA computes the same table of range starts once.
    int* s_lo = (int*)(smem + L.lo_off);
    const unsigned* s_pv = (const unsigned*)(smem + L.pv_off);
    const float rG = __frcp_rz(__int2float_rz(G));
    if constexpr (kCompact) {
        if (alive && wsplit) {
            // this CTA's own four range ends, one warp each (two 32-way steps find the virtual expert: U <= 1024);
            // the accumulator warps fill in the other CTAs' while the first weight tiles are in flight
            if (warp < 4) {
                const int ph = warp >> 1, c = cta + (warp & 1);
                const unsigned* p1 = s_pv + ph * L.pv_stride;
                const int n_u = ph ? HB * KBd : IB * KBu;
                int lo_ks = U * n_u;
                if (c < G) {
                    const unsigned target = split_target(p1[U], c, rG);
                    const int stride = (U + 31) >> 5;
                    const int b1 = __popc(__ballot_sync(0xffffffffu, lane * stride < U && p1[lane * stride] <= target)) - 1;   // p1[0] = 0
                    const int i2 = b1 * stride + lane;
                    const int a = b1 * stride + __popc(__ballot_sync(0xffffffffu, lane < stride && i2 < U && p1[i2] <= target)) - 1;
                    lo_ks = split_point(p1, a, target, n_u, ph ? KBd : KBu, ph ? q_dn : q_up);
                }
                if (lane == 0) s_lo[ph * (kMaxGrid + 1) + c] = lo_ks;
            }
            __syncthreads();
        }
    }
    auto rlo = [&](int ph, int c) -> int {
        if constexpr (kCompact) { if (wsplit) return s_lo[ph * (kMaxGrid + 1) + c]; }
        return ph ? range_lo(Sq_dn, c, q_dn, gm) : range_lo(Sq_up, c, q_up, gm);
    };
    const int up_lo = alive ? rlo(0, cta) : 0, up_hi = alive ? rlo(0, cta + 1) : 0;
    const int dn_lo = alive ? rlo(1, cta) : 0, dn_hi = alive ? rlo(1, cta + 1) : 0;

    // ------------------------------------------------------------------ role: TMA producers
    // Stage sequence: an up k-step contributes two stages (gate tile, up tile), a down k-step one.  A stage = one
    // 128x128 weight tile (warp 0) + one Nx128 activation tile (warp 2), each on its own mbarrier; the up tile of a
    // k-step reuses the activation tile of its gate stage.  Two issuing threads because one thread cannot issue
    // two bulk-tensor copies per 16 KiB fast enough to saturate HBM3e; and because only the activation tiles of the
    // down projection wait for the up projection's intermediate tile, the weight stream never stalls on it
    // (Section 3.3: lookahead across the projection boundary).
    if (warp == 0) {
        if (lane == 0 && alive) {
            const uint64_t stream_once = l2_policy_evict_first();
            const int n_up_st = 2 * (up_hi - up_lo), n_st = n_up_st + (dn_hi - dn_lo);
            Walk aw;
            int a_cur = 0, a_st = 0;
            uint32_t a_ph = 1u;                  // parity to wait for on the empty barrier
            uint32_t dst = smem_u32(smem), full = bar_full, empty = bar_empty;
            if (n_up_st > 0) aw.init(up_lo, KBu, IB, s_act);
            else if (n_st > 0) aw.init(dn_lo, KBd, HB, s_act);
            bool stamped = false;
            MOE_STAMP_ALWAYS(8);
            for (; a_cur < n_up_st; ++a_cur) {                       // gate/up weight tiles
                if (!wt.mbar(empty, a_ph, 2)) break;
                const int half = a_cur & 1;
                mbar_expect_tx(full, (uint32_t)kATileBytes);
                tma_load_2d_hint(dst, &tmW13, aw.kb * kBlock, (aw.e & 0xFFFF) * 2 * I + half * I + aw.mb * kBlock, full, stream_once);
                if (half) aw.next(s_act);
                dst += L.stage_bytes; full += 8; empty += 8;
                if (++a_st == S) { a_st = 0; a_ph ^= 1u; dst = smem_u32(smem); full = bar_full; empty = bar_empty; if (!stamped) { MOE_STAMP_ALWAYS(9); stamped = true; } }
            }
            if (!wt.dead && n_st > n_up_st) aw.init(dn_lo, KBd, HB, s_act);
            for (; a_cur < n_st && !wt.dead; ++a_cur) {              // down weight tiles
                if (!wt.mbar(empty, a_ph, 2)) break;
                mbar_expect_tx(full, (uint32_t)kATileBytes);
                tma_load_2d_hint(dst, &tmW2, aw.kb * kBlock, (aw.e & 0xFFFF) * H + aw.mb * kBlock, full, stream_once);
                aw.next(s_act);
                dst += L.stage_bytes; full += 8; empty += 8;
                if (++a_st == S) { a_st = 0; a_ph ^= 1u; dst = smem_u32(smem); full = bar_full; empty = bar_empty; }
            }
            misc[6] = (uint32_t)a_cur;      // weight tiles requested (the teardown waits for them if the launch gave up)
        }
        __syncwarp();
    }
    else if (warp == 2 && kCompact) {
        // Compacted tokens: the activation tile of an up k-step is gathered -- row r = the quantised input of the
        // unit's r-th token -- by the whole warp with 16-byte asynchronous copies into the 128-byte-swizzled layout
        // the MMA expects (chunk c of row r sits at chunk c ^ (r & 7)); every lane arrives on the stage's barrier
        // once its copies have landed.  The down projection's tile is one bulk-tensor copy (rows are already compact).
        if (alive) {
            const int n_up_st = 2 * (up_hi - up_lo), n_st = n_up_st + (dn_hi - dn_lo);
            Walk bw;
            int b_cur = 0, b_st = 0;
            uint32_t b_ph = 1u;
            uint32_t dst = smem_u32(smem) + kATileBytes, full = bar_fullb, empty = bar_empty;
            if (n_up_st > 0) bw.init(up_lo, KBu, IB, s_act);
            else if (n_st > 0) bw.init(dn_lo, KBd, HB, s_act);
            const int chunk = lane & 7, r0 = lane >> 3;          // this lane copies chunk `chunk` of rows r0, r0+4, r0+8, ...
            int b_entry = -1;
            int tokr[N / 4];
#pragma unroll
            for (int i = 0; i < N / 4; ++i) tokr[i] = -1;
            bool ok = true;
            for (; b_cur < n_up_st; ++b_cur) {
                if (lane == 0) ok = wt.mbar(empty, b_ph, 10);
                ok = __shfl_sync(0xffffffffu, ok, 0);
                if (!ok) break;
                if ((b_cur & 1) == 0) {
                    if (bw.e != b_entry) {
                        b_entry = bw.e;
                        const TokMask m = load_mask(s_mask, b_entry & 0xFFFF);
                        const int colbase = (b_entry >> 16) * N, cnt = min(N, mask_count(m) - colbase);
#pragma unroll
                        for (int i = 0; i < N / 4; ++i) tokr[i] = (r0 + 4 * i < cnt) ? mask_nth(m, colbase + r0 + 4 * i) : -1;
                    }
#pragma unroll
                    for (int i = 0; i < N / 4; ++i) {
                        const int r = r0 + 4 * i;
                        if (tokr[i] >= 0)
                            cp_async16(dst + (uint32_t)(r * kBlock + ((chunk ^ (r & 7)) << 4)),
                                       P.xq + (size_t)tokr[i] * H + bw.kb * kBlock + chunk * 16);
                    }
                    cp_async_mbar_arrive(full);
                } else {
                    mbar_arrive(full);
                    bw.next(s_act);
                }
                dst += L.stage_bytes; full += 8; empty += 8;
                if (++b_st == S) { b_st = 0; b_ph ^= 1u; dst = smem_u32(smem) + kATileBytes; full = bar_fullb; empty = bar_empty; }
            }
            if (ok && n_st > n_up_st) bw.init(dn_lo, KBd, HB, s_act);
            int ready_e = -1;                    // unit whose intermediate tile is known to be published
            for (; b_cur < n_st && ok; ++b_cur) {
                if (lane == 0) ok = wt.mbar(empty, b_ph, 10);
                ok = __shfl_sync(0xffffffffu, ok, 0);
                if (!ok) break;
                const int be = bw.e & 0xFFFF, bpass = bw.e >> 16;
                if (bw.e != ready_e) {                               // published? (Section 3.2, readiness hand-off)
                    if (lane == 0) { ok = wt.flag(e_cnt + bpass * E + be, (unsigned)IB, 11); fence_proxy_async(); }
                    ok = __shfl_sync(0xffffffffu, ok, 0);
                    if (!ok) break;
                    ready_e = bw.e;
                }
                if (lane == 0) {
                    mbar_expect_tx(full, (uint32_t)(N * kBlock));
                    tma_load_2d(dst, &tmHq, bw.kb * kBlock, be * P.nr + bpass * N, full);
                } else {
                    mbar_arrive(full);
                }
                bw.next(s_act);
                dst += L.stage_bytes; full += 8; empty += 8;
                if (++b_st == S) { b_st = 0; b_ph ^= 1u; dst = smem_u32(smem) + kATileBytes; full = bar_fullb; empty = bar_empty; }
            }
            cp_async_wait_all();                 // nothing of this warp is in flight past this point, except bulk copies:
            if (lane == 0) misc[7] = (uint32_t)b_cur;   // activation tiles requested (the teardown waits for them if the launch gave up)
        }
        __syncwarp();
    }
    else if (warp == 2) {
        if (lane == 0 && alive) {
            fence_proxy_async();                 // xq was written with ordinary stores by other CTAs
            const int n_up_st = 2 * (up_hi - up_lo), n_st = n_up_st + (dn_hi - dn_lo);
            Walk bw;
            int b_cur = 0, b_st = 0;
            uint32_t b_ph = 1u;
            uint32_t dst = smem_u32(smem) + kATileBytes, full = bar_fullb, empty = bar_empty;
            if (n_up_st > 0) bw.init(up_lo, KBu, IB, s_act);
            else if (n_st > 0) bw.init(dn_lo, KBd, HB, s_act);
            for (; b_cur < n_up_st; ++b_cur) {                       // input activation tiles (gate stages only)
                if (!wt.mbar(empty, b_ph, 10)) break;
                if ((b_cur & 1) == 0) {
                    mbar_expect_tx(full, (uint32_t)(N * kBlock));
                    tma_load_2d(dst, &tmXq, bw.kb * kBlock, 0, full);
                } else {
                    mbar_arrive(full);
                    bw.next(s_act);
                }
                dst += L.stage_bytes; full += 8; empty += 8;
                if (++b_st == S) { b_st = 0; b_ph ^= 1u; dst = smem_u32(smem) + kATileBytes; full = bar_fullb; empty = bar_empty; }
            }
            if (!wt.dead && n_st > n_up_st) bw.init(dn_lo, KBd, HB, s_act);
            int ready_e = -1;                    // expert whose intermediate tile is known to be published
            for (; b_cur < n_st && !wt.dead; ++b_cur) {              // intermediate activation tiles
                if (!wt.mbar(empty, b_ph, 10)) break;
                const int be = bw.e & 0xFFFF, bpass = bw.e >> 16;
                if (bw.e != ready_e) {                               // published? (Section 3.2, readiness hand-off)
                    if (!wt.flag(e_cnt + bpass * E + be, (unsigned)IB, 11)) break;
                    fence_proxy_async();
                    ready_e = bw.e;
                }
                mbar_expect_tx(full, (uint32_t)(N * kBlock));
                tma_load_2d(dst, &tmHq, bw.kb * kBlock, be * P.nr + bpass * N, full);
                bw.next(s_act);
                dst += L.stage_bytes; full += 8; empty += 8;
                if (++b_st == S) { b_st = 0; b_ph ^= 1u; dst = smem_u32(smem) + kATileBytes; full = bar_fullb; empty = bar_empty; }
            }
            misc[7] = (uint32_t)b_cur;      // activation tiles requested (the teardown waits for them if the launch gave up)
        }
        __syncwarp();
    }
    // ------------------------------------------------------------------ role: MMA issuers
    // Two issuing threads (warp 1: even k-steps, warp 3: odd k-steps), each with its own TMEM buffers (k-step mod 8)
    // and its own commits: issuing four tcgen05.mma per 16 KiB tile from one thread alone costs more time than the
    // tile takes to arrive from HBM.
    // The two share the stage ring, and a stage's previous user may have been the other issuer.  A parity wait cannot
    // tell "my phase is complete" from "the phase before the previous one is complete", so an issuer that runs ahead
    // (tiles land out of order) must not wait on a stage whose previous phase the other issuer has not seen complete:
    // each publishes the number of k-steps it has issued, and nobody gets S/2 or more k-steps ahead of the other (a
    // lap of the ring is at least S/2 k-steps, so the previous user of any of my stages is then done with them).
    else if (warp == 1 || warp == 3) {
        if (lane == 0 && alive) {
            constexpr uint32_t idesc = (1u << 4) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(kBlock >> 4) << 24);
            const uint32_t ring = smem_u32(smem);
            const int who = warp >> 1;           // 0 or 1
            const int n_up = up_hi - up_lo, n_dn = dn_hi - dn_lo;
            int st = 0;
            uint32_t ph = 0;                     // full-barrier parity of stage `st`
            auto advance = [&](int n) { st += n; while (st >= S) { st -= S; ph ^= 1u; } };
            bool first = true;
            int other_seen = 0;                  // k-steps the other issuer was last seen to have issued
            if (who == 1) advance(n_up > 0 ? 2 : 1);               // skip k-step 0
            for (int ks = who; ks < n_up + n_dn && !wt.dead; ks += 2) {
                const bool up = ks < n_up;
                const int buf = ks & (kTmemBufs - 1);
                const uint32_t tph = (uint32_t)((ks >> kBufShift) & 1) ^ 1u;
                if (!wt.mbar(bar_tempty + 8 * buf, tph, 3)) break;
                {
                    // the other issuer's k-steps up to q = ks - S/2 must be issued: the last of them is q or q - 1
                    const int q = ks - (S >> 1);
                    const int thr = ((q & 1) != who) ? q + 1 : q;                      // its progress count once that one is issued
                    if (other_seen < thr) {                                             // (re-read only when the cached count is too old)
                        volatile uint32_t* other = misc + 4 + (who ^ 1);
                        bool ok = true;
                        for (uint32_t i = 1; (other_seen = (int)*other) < thr; ++i)
                            if ((i & 255u) == 0 && wt.expired(13)) { ok = false; break; }
                        if (!ok) break;
                    }
                }
                const int st0 = st;
                const uint32_t ph0 = ph;
                const uint32_t a0 = ring + (uint32_t)st0 * (uint32_t)L.stage_bytes;
                if (!wt.mbar(bar_full + 8 * st0, ph0, 4) || !wt.mbar(bar_fullb + 8 * st0, ph0, 4)) break;
                if (kCompact && up) fence_proxy_async();       // the gathered tile was written through the generic proxy
                const uint64_t b_desc = make_smem_desc(a0 + kATileBytes);
                const uint32_t d = tmem_base + (uint32_t)(buf * 2 * N);
                if (first && who == 0) { MOE_STAMP_ALWAYS(10); first = false; }
                tc_fence_after();
                {
                    const uint64_t a_desc = make_smem_desc(a0);
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        umma_f8(d, a_desc + (uint64_t)(k * 2), b_desc + (uint64_t)(k * 2), idesc, k > 0 ? 1u : 0u);
                }
                if (up) {                                      // up tile of the same K block, same activation tile
                    advance(1);
                    const int st1 = st;
                    if (!wt.mbar(bar_full + 8 * st1, ph, 4) || !wt.mbar(bar_fullb + 8 * st1, ph, 4)) break;
                    tc_fence_after();
                    const uint64_t a_desc = make_smem_desc(ring + (uint32_t)st1 * (uint32_t)L.stage_bytes);
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        umma_f8(d + N, a_desc + (uint64_t)(k * 2), b_desc + (uint64_t)(k * 2), idesc, k > 0 ? 1u : 0u);
                    umma_commit(bar_empty + 8 * st0);          // both stages reusable once all eight MMAs retire
                    umma_commit(bar_empty + 8 * st1);
                } else {
                    umma_commit(bar_empty + 8 * st0);
                }
                umma_commit(bar_tfull + 8 * buf);              // accumulator of this K block complete
                *(volatile uint32_t*)(misc + 4 + who) = (uint32_t)(ks + 1);     // every k-step below ks + 1 of mine is issued
                // move past the rest of this k-step and the other issuer's k-step
                advance(1);
                if (ks + 1 < n_up + n_dn) advance(ks + 1 < n_up ? 2 : 1);
            }
        }
        __syncwarp();
    }
    // ------------------------------------------------------------------ role: accumulator / epilogue warps
    else if (warp >= kEpiWarp0 && alive) {
        const int q = warp & 3, row = q * 32 + lane;           // TMEM lane == weight row inside the tile
        const int etid = tid - kEpiWarp0 * 32;
        const int cb = ((warp - kEpiWarp0) >> 2) * TCG;        // first token column of this accumulator group
        // column of register slot n: the group's columns in order -- except in the 32-column compacted variant, where
        // the two groups take alternating blocks of 8 columns: the columns in use are the first `cnt`, and this way both
        // groups share them (slots in use stay contiguous from 0: a group's second block fills only after its first)
        constexpr bool kInterleave = kCompact && kEpiGroups == 2;
        auto colx = [&](int n) -> int { return kInterleave ? ((n & 8) << 1) + (cb >> 1) + (n & 7) : cb + n; };
        const uint32_t t_lane = tmem_base + ((uint32_t)(q * 32) << 16);
        volatile uint32_t* s_giveup = misc + 3;
        bool first_acc = true;
        constexpr int CH = kCompact ? 4 : (TCG < 16 ? TCG : 16);   // columns per TMEM load
        int buf = 0, hs_e = -1;
        uint32_t tph = 0;
        float accg[TCG], accu[TCG];
        // columns of the current (expert, pass): token set (first word), columns in use, and per lane the token and
        // the y row of column colx(lane)
        int col_entry = -1, cnt = TCG, tok_lane = colx(lane), yoff_lane = 0;
        unsigned long long mask = 0ull;
        auto col_on = [&](int n) -> bool { return kCompact ? (colx(n) < cnt) : (bool)((mask >> (colx(n))) & 1ull); };

        // The routed (token, slot) pairs grouped by expert, tokens ascending -- entry r of expert e is the r-th token
        // routed to e and the top-k slot e holds for it.  The compacted variants need it from the first up unit on and
        // build it while the first weight tiles are in flight; the others only need it for the down projection and
        // build it while they wait for the first intermediate tile to be published.
        auto build_pairs = [&]() {
        if (warp == kEpiWarp0) {
            int base = 0;
#pragma unroll 1
            for (int e0 = 0; e0 < E; e0 += 32) {
                const int c = (e0 + lane < E) ? mask_count(load_mask(s_mask, e0 + lane)) : 0;
                int incl = c;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) { const int v = __shfl_up_sync(0xffffffffu, incl, o); if (lane >= o) incl += v; }
                if (e0 + lane < E) s_poff[e0 + lane] = base + incl - c;
                base += __shfl_sync(0xffffffffu, incl, 31);
            }
        }
        epi_bar(kEpiThreads);
#pragma unroll 1
        for (int pi = etid; pi < T * K; pi += kEpiThreads) {
            const int t = div_small(pi, K), ex = s_ids[pi];
            s_pair[s_poff[ex] + mask_rank(load_mask(s_mask, ex), t)] = (unsigned short)(t | ((pi - t * K) << 8));
        }
        epi_bar(kEpiThreads);
        };
        if constexpr (kCompact) {
            if (wsplit) {                                  // every CTA's range starts (ordered before their first use by build_pairs' barriers)
#pragma unroll 1
                for (int i = etid; i < 2 * (G + 1); i += kEpiThreads) {
                    const int ph = (i > G) ? 1 : 0, c = i - ph * (G + 1);
                    const unsigned* p1 = s_pv + ph * L.pv_stride;
                    const int n_u = ph ? HB * KBd : IB * KBu;
                    int lo_ks = U * n_u;
                    if (c < G) {
                        const unsigned target = split_target(p1[U], c, rG);
                        int a = 0, b = U - 1;              // largest u with p1[u] <= target
                        while (a < b) { const int m = (a + b + 1) >> 1; if (p1[m] <= target) a = m; else b = m - 1; }
                        lo_ks = split_point(p1, a, target, n_u, ph ? KBd : KBu, ph ? q_dn : q_up);
                    }
                    s_lo[ph * (kMaxGrid + 1) + c] = lo_ks;
                }
            }
            build_pairs();
        }

        for (int phase = 0; phase < 2 && !wt.dead; ++phase) {
            const bool up = (phase == 0);
            const int lo = up ? up_lo : dn_lo, hi = up ? up_hi : dn_hi;
            const int KB = up ? KBu : KBd, MB = up ? IB : HB;  // K blocks per unit, row blocks per expert
            const int rph = up ? 0 : 1;
            float* part = up ? P.part_up : P.part_dn;
            unsigned* pflag = up ? P.pu_flag : P.pd_flag;
            const int pcols = up ? 2 * N : N;
            if (!up && etid == 0) MOE_STAMP_ALWAYS(12);
            if (hi <= lo) continue;
            if (!kCompact && !up) { build_pairs(); col_entry = -1; }
            Walk w;
            w.init(lo, KB, MB, s_act);

            // Block scales of the weight tiles: lane l of every warp holds the scales of k-step (32*block + l) of
            // this CTA's range and hands them out by shuffle; the next block of 32 is fetched one block ahead.
            auto fetch_scales = [&](int sidx, float& g, float& u2) {
                g = 0.f; u2 = 0.f;
                if (sidx < hi) {
                    const int unit = div_small(sidx, KB), kb = sidx - unit * KB, uu = div_small(unit, MB), mb = unit - uu * MB, e = s_act[uu] & 0xFFFF;
                    if (up) {
                        g = __ldg(P.W13s + ((size_t)e * 2 * IB + mb) * KBu + kb);
                        u2 = __ldg(P.W13s + ((size_t)e * 2 * IB + IB + mb) * KBu + kb);
                    } else {
                        g = __ldg(P.W2s + ((size_t)e * HB + mb) * KBd + kb);
                    }
                }
            };
            float sg_cur, su_cur, sg_nxt, su_nxt;
            fetch_scales(lo + lane, sg_cur, su_cur);
            fetch_scales(lo + 32 + lane, sg_nxt, su_nxt);

            for (int s = lo; s < hi && !wt.dead;) {
                // ---- one piece: the k-steps [s, pend) of unit (e, mb), first K block kb0
                const int entry = w.e, e = entry & 0xFFFF, colbase = (entry >> 16) * N, mb = w.mb, kb0 = w.kb;
                const int ustart = s - kb0, uend = ustart + KB;
                const int pend = uend < hi ? uend : hi;
                // lane l of every warp looks after column cb + l: its token and (down projection) where its result goes;
                // consecutive units of a range mostly belong to the same (expert, pass), whose columns are kept
                if (entry != col_entry) {
                    col_entry = entry;
                    mask = s_mask[2 * e];                      // tokens 0..63 (all there are unless compacted)
                    cnt = TCG; tok_lane = colx(lane); yoff_lane = 0;
                    if constexpr (kCompact) cnt = min(N, __popcll(mask) + __popcll(s_mask[2 * e + 1]) - colbase);
                    if ((kCompact || !up) && lane < TCG && col_on(lane)) {
                        const int r = kCompact ? colbase + colx(lane) : __popcll(mask & ((1ull << (colx(lane))) - 1ull));
                        const unsigned pr = s_pair[s_poff[e] + r];
                        tok_lane = (int)(pr & 0xFFu);
                        yoff_lane = (tok_lane * K + (int)(pr >> 8)) * H;   // first element of the (token, slot) row of y
                    }
                }
                if (!up && entry != hs_e) {
                    // activation scales of this expert's intermediate tile -> shared memory (once per expert and pass)
                    const bool got = (etid == 0) ? wt.flag(e_cnt + (entry >> 16) * E + e, (unsigned)IB, 8) : true;
                    if (!epi_all(got, kEpiThreads)) { wt.dead = true; break; }
                    for (int i = etid; i < IB * N; i += kEpiThreads) s_hs[i] = __ldcg(P.hs + ((size_t)e * IB + i / N) * P.nr + colbase + i % N);
                    hs_e = entry;
                    epi_bar(kEpiThreads);
                }
                if constexpr (kCompact) {
                    if (up) {
                        // input scales of this piece's K blocks, gathered for the unit's tokens: [K block][column]
                        if (q == 0 && lane < TCG) s_utok[colx(lane)] = tok_lane;   // each group's first warp: its columns
                        epi_bar(kEpiThreads);
                        for (int idx = etid; idx < (pend - s) * N; idx += kEpiThreads) {
                            const int c = idx & (N - 1);
                            s_as[idx] = (c < cnt) ? s_xs[(kb0 + idx / N) * TS + s_utok[c]] : 0.f;
                        }
                        epi_bar(kEpiThreads);
                    }
                }
                const float* as_p = up ? (kCompact ? s_as : s_xs + kb0 * TS) : (s_hs + kb0 * N);   // activation scales [K block][column]
                const int as_step = up ? (kCompact ? N : TS) : N;
#pragma unroll
                for (int n = 0; n < TCG; ++n) { accg[n] = 0.f; accu[n] = 0.f; }

                // Two k-steps per turn when the second accumulator is already complete (one warp per scheduler: nothing
                // else hides the TMEM-load latency); one k-step otherwise, so a just-in-time MMA stream is never waited on.
                constexpr bool kDual = (TCG <= 16) && !kCompact;
                auto next_scales = [&](int sidx, float& g, float& u2) {
                    const int j = (sidx - lo) & 31;
                    if (j == 0 && sidx != lo) {
                        sg_cur = sg_nxt; su_cur = su_nxt;
                        fetch_scales(sidx + 32 + lane, sg_nxt, su_nxt);
                    }
                    g = __shfl_sync(0xffffffffu, sg_cur, j);
                    u2 = __shfl_sync(0xffffffffu, su_cur, j);
                };
                auto load_acc = [&](int b, float* dg, float* du) {
                    const uint32_t tcol = t_lane + (uint32_t)(b * 2 * N);
                    if constexpr (kCompact) {
                        // one load as wide as the routed columns need (warp-uniform): a TMEM load costs about the
                        // same whatever its width
                        // slots in use: the group's columns below cnt
                        const int need = kInterleave ? min(8, max(0, cnt - (cb >> 1))) + min(8, max(0, cnt - 16 - (cb >> 1))) : cnt - cb;
                        if (need <= 4) {
                            tmem_ld<4>(tcol + colx(0), dg);
                            if (up) tmem_ld<4>(tcol + N + colx(0), du);
                        } else if (need <= 8) {
                            tmem_ld<8>(tcol + colx(0), dg);
                            if (up) tmem_ld<8>(tcol + N + colx(0), du);
                        } else if constexpr (kInterleave) {
                            tmem_ld<8>(tcol + colx(0), dg);
                            tmem_ld<8>(tcol + colx(8), dg + 8);
                            if (up) { tmem_ld<8>(tcol + N + colx(0), du); tmem_ld<8>(tcol + N + colx(8), du + 8); }
                        } else {
                            tmem_ld<16>(tcol + colx(0), dg);
                            if (up) tmem_ld<16>(tcol + N + colx(0), du);
                        }
                    } else {
#pragma unroll
                        for (int c = 0; c < TCG; c += CH) {
                            tmem_ld<CH>(tcol + colx(c), dg + c);
                            if (up) tmem_ld<CH>(tcol + N + colx(c), du + c);
                        }
                    }
                };
                auto add_scaled = [&](const float* dg, const float* du, float wsg, float wsu, int i) {
#pragma unroll
                    for (int c = 0; c < TCG; c += CH) {
                        if (kCompact && colx(c) >= cnt) break;
                        float as[CH];
                        if constexpr (CH >= 4) {
#pragma unroll
                            for (int jj = 0; jj < CH; jj += 4) {
                                const float4 v = *reinterpret_cast<const float4*>(as_p + i * as_step + colx(c) + jj);
                                as[jj] = v.x; as[jj + 1] = v.y; as[jj + 2] = v.z; as[jj + 3] = v.w;
                            }
                        } else {
#pragma unroll
                            for (int jj = 0; jj < CH; ++jj) as[jj] = as_p[i * as_step + colx(c) + jj];
                        }
#pragma unroll
                        for (int jj = 0; jj < CH; ++jj) {
                            const int n = c + jj;
                            accg[n] = fmaf(dg[n], wsg * as[jj], accg[n]);
                            if (up) accu[n] = fmaf(du[n], wsu * as[jj], accu[n]);
                        }
                    }
                };
                for (int i = 0; i < pend - s;) {
                    float wsg0, wsu0, wsg1 = 0.f, wsu1 = 0.f;
                    next_scales(s + i, wsg0, wsu0);
                    // A wait that runs out is recorded and the warp keeps walking in lockstep with the others;
                    // the piece end below turns the record into a uniform decision to stop.
                    if (!wt.mbar(bar_tfull + 8 * buf, tph, 5)) *s_giveup = 1u;
                    int buf1 = buf + 1;
                    uint32_t tph1 = tph;
                    if (buf1 == kTmemBufs) { buf1 = 0; tph1 ^= 1u; }
                    bool two = false;
                    if constexpr (kDual)
                        two = (i + 1 < pend - s) && __all_sync(0xffffffffu, mbar_try_wait(bar_tfull + 8 * buf1, tph1));
                    if (two) next_scales(s + i + 1, wsg1, wsu1);
                    tc_fence_after();
                    if (first_acc) { if (etid == 0) MOE_STAMP_ALWAYS(11); first_acc = false; }
                    // all TMEM loads first, one wait, free the buffers, then the arithmetic
                    float dg0[TCG], du0[TCG], dg1[kDual ? TCG : 1], du1[kDual ? TCG : 1];
                    load_acc(buf, dg0, du0);
                    if constexpr (kDual) { if (two) load_acc(buf1, dg1, du1); }
                    tmem_ld_wait();
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) { mbar_arrive(bar_tempty + 8 * buf); if (two) mbar_arrive(bar_tempty + 8 * buf1); }
                    add_scaled(dg0, du0, wsg0, wsu0, i);
                    if constexpr (kDual) { if (two) add_scaled(dg1, du1, wsg1, wsu1, i + 1); }
                    if (two) { buf = buf1; tph = tph1; ++i; }
                    ++i;
                    if (++buf == kTmemBufs) { buf = 0; tph ^= 1u; }
                }
                const bool unit_done = (pend == uend);
                s = pend;
                if (unit_done) w.next_unit(s_act);
                if (!up && unit_done && ustart >= lo) {
                    // whole down unit: every warp stores its rows and counts itself done -- no block-level barrier
                    // (units of the down projection can be as short as two k-steps)
#pragma unroll
                    for (int n = 0; n < TCG; ++n) {
                        if (kCompact && colx(n) >= cnt) break;               // compacted columns are contiguous: stop at the first unused one
                        if (col_on(n)) {
                            const int yo = __shfl_sync(0xffffffffu, yoff_lane, n);
                            __stcg(P.y + (size_t)yo + mb * kBlock + row, accg[n]);
                        }
                    }
                    continue;                                   // published once per CTA, after the last down unit
                }
                epi_bar(kEpiThreads);
                if (*s_giveup) { wt.dead = true; break; }

                // ---- end of this CTA's piece of the unit: combine split-K partials, then the epilogue
                if (ustart < lo) {
                    // not the owner: park the partial accumulator, [column][row] so rows are contiguous
                    float* dst = part + (size_t)cta * pcols * kBlock;
#pragma unroll
                    for (int n = 0; n < TCG; ++n) {
                        if (kCompact && colx(n) >= cnt) break;               // compacted columns are contiguous: stop at the first unused one
                        if (col_on(n)) {                        // only tokens routed to this expert matter
                            __stcg(dst + (colx(n)) * kBlock + row, accg[n]);
                            if (up) __stcg(dst + (N + colx(n)) * kBlock + row, accu[n]);
                        }
                    }
                    epi_bar(kEpiThreads);
                    if (etid == 0) st_release(pflag + cta, tag);
                    continue;
                }
                if (!unit_done) {
                    // owner of a unit that continues in later CTAs: wait for all of them at once (one thread per
                    // contributor), then add their partials in CTA order
                    int c_end = cta + 1;
                    bool got = true;
                    for (int base = cta + 1; base < G; base += kEpiThreads) {
                        const int c = base + etid;
                        if (c < G) {
                            const int clo = rlo(rph, c), chi = rlo(rph, c + 1);
                            if (clo < uend && chi > clo) got = wt.flag(pflag + c, tag, 6) && got;
                        }
                        if (rlo(rph, min(base + kEpiThreads, G)) >= uend) break;
                    }
                    while (c_end < G && rlo(rph, c_end) < uend) ++c_end;
                    if (!epi_all(got, kEpiThreads)) { wt.dead = true; break; }
                    for (int c = cta + 1; c < c_end; ++c) {
                        if (rlo(rph, c + 1) == rlo(rph, c)) continue;
                        const float* src = part + (size_t)c * pcols * kBlock;
#pragma unroll
                        for (int n = 0; n < TCG; ++n) {
                            if (kCompact && colx(n) >= cnt) break;               // compacted columns are contiguous: stop at the first unused one
                            if (col_on(n)) {
                                accg[n] += __ldcg(src + (colx(n)) * kBlock + row);
                                if (up) accu[n] += __ldcg(src + (N + colx(n)) * kBlock + row);
                            }
                        }
                    }
                }
                if (up) {
                    // SiLU(gate)*up, 128-wide amax, FP8 requantisation, one global store  (Section 3.3)
#pragma unroll
                    for (int n = 0; n < TCG; ++n) {
                        if (kCompact && colx(n) >= cnt) break;               // compacted columns are contiguous: stop at the first unused one
                        if (col_on(n)) {                        // warp-uniform: other tokens cost nothing
                            const float g = accg[n];
                            const float a = __fdiv_rn(g, 1.0f + expf(-g)) * accu[n];
                            accg[n] = a;
                            // |a| as an integer orders like the float: one warp-wide integer max instead of a shuffle tree
                            const uint32_t m = __reduce_max_sync(0xffffffffu, __float_as_uint(fabsf(a)));
                            if (lane == 0) s_red[q * N + colx(n)] = __uint_as_float(m);
                        }
                    }
                    epi_bar(kEpiThreads);
#pragma unroll
                    for (int n = 0; n < TCG; ++n) {
                        if (kCompact && colx(n) >= cnt) break;               // compacted columns are contiguous: stop at the first unused one
                        if (col_on(n)) {
                            const float amax = fmaxf(fmaxf(s_red[colx(n)], s_red[N + colx(n)]), fmaxf(s_red[2 * N + colx(n)], s_red[3 * N + colx(n)]));
                            const float sc = __fdiv_rn(fmaxf(amax, 1e-10f), 448.0f);
                            const float2 v = make_float2(__fdiv_rn(accg[n], sc), 0.f);
                            const uint8_t code = (uint8_t)(__nv_cvt_float2_to_fp8x2(v, __NV_SATFINITE, __NV_E4M3) & 0xFF);
                            P.hq[((size_t)e * P.nr + colbase + colx(n)) * I + mb * kBlock + row] = code;
                            if (row == 0) P.hs[((size_t)e * IB + mb) * P.nr + colbase + colx(n)] = sc;
                        }
                    }
                    fence_proxy_async();
                    epi_bar(kEpiThreads);
                    if (etid == 0) red_release_add(e_cnt + (entry >> 16) * E + e, 1u);   // the expert's tile (of this pass) is complete at count == I/128
                } else {
                    // per-slot result of this expert for its routed tokens
#pragma unroll
                    for (int n = 0; n < TCG; ++n) {
                        if (kCompact && colx(n) >= cnt) break;               // compacted columns are contiguous: stop at the first unused one
                        if (col_on(n)) {
                            const int yo = __shfl_sync(0xffffffffu, yoff_lane, n);
                            __stcg(P.y + (size_t)yo + mb * kBlock + row, accg[n]);
                        }
                    }
                    // (published once per CTA, after the last down unit)
                }
            }
        }
        // every down-projection result of this CTA's range is stored: one release for all of them (a release per
        // unit would stall on the unit's own stores; units can be as short as two k-steps)
        epi_bar(kEpiThreads);
        if (etid == 0) { st_release(P.dn_flag + cta, tag); MOE_STAMP_ALWAYS(13); }
        // ---- final weighted reduction in slot order (deterministic); tasks (token, 128-row block): task = cta + i * G.
        // First every (task, slot) of this CTA waits for the CTA that stored its down-projection result -- all of
        // them in parallel, one thread each -- then the tasks are summed two (four for 16 token columns and more) at a time so that their loads overlap.
        const int grp = (warp - kEpiWarp0) >> 2;
        const int n_tasks = T * HB, n_mine = (cta < n_tasks) ? (n_tasks - cta + G - 1) / G : 0;
        {
            bool got = true;
#pragma unroll 1
            for (int idx = etid; idx < n_mine * K; idx += kEpiThreads) {
                const int i = div_small(idx, K), j = idx - i * K, task = cta + i * G;
                const int t = div_small(task, HB), hb = task - t * HB;
                // the CTA that owns unit (expert, hb) of the down projection = the one whose range holds its first k-step
                const int ex = s_ids[t * K + j];
                const int ps = kCompact ? mask_rank(load_mask(s_mask, ex), t) / N : 0;   // the pass that holds token t
                const unsigned unit = (unsigned)((s_uidx[ex] + ps) * HB + hb);
                unsigned owner;
                if (kCompact && wsplit) {
                    const int xk = (int)unit * KBd;                                    // first k-step of the unit
                    int a = 0, b = G - 1;                                              // the CTA whose range holds it
                    while (a < b) { const int m = (a + b + 1) >> 1; if (rlo(1, m) <= xk) a = m; else b = m - 1; }
                    owner = (unsigned)a;
                } else {
                    const unsigned x = (q_dn == 1) ? unit * (unsigned)KBd : unit;      // first quantum of the unit
                    owner = ((x + 1u) * (unsigned)G - 1u) / (unsigned)Sq_dn;
                }
                got = wt.flag(P.dn_flag + owner, tag, 7) && got;
            }
            if (!epi_all(got, kEpiThreads)) wt.dead = true;
        }
        constexpr int RT = (TC >= 16) ? 4 : 2;                 // tasks summed together: RT x 8 loads in flight per thread
        for (int i0 = grp; i0 < n_mine && !wt.dead; i0 += RT * kEpiGroups) {
            int tt[RT], hh[RT];
            const float* yp[RT];
            float acc[RT];
#pragma unroll
            for (int r = 0; r < RT; ++r) {
                const int i = i0 + r * kEpiGroups;
                const int task = cta + (i < n_mine ? i : i0) * G;  // (absent tasks repeat the first: loads stay legal, nothing is stored)
                tt[r] = div_small(task, HB);
                hh[r] = task - tt[r] * HB;
                yp[r] = P.y + (size_t)tt[r] * K * H + hh[r] * kBlock + row;
                acc[r] = 0.f;
            }
            for (int j0 = 0; j0 < K; j0 += 8) {
                float v[RT][8];
#pragma unroll
                for (int r = 0; r < RT; ++r)
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        v[r][j] = (j0 + j < K && i0 + r * kEpiGroups < n_mine) ? __ldcg(yp[r] + (size_t)(j0 + j) * H) : 0.f;
#pragma unroll
                for (int r = 0; r < RT; ++r)
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        if (j0 + j < K) acc[r] = fmaf(s_w[tt[r] * K + j0 + j], v[r][j], acc[r]);
            }
#pragma unroll
            for (int r = 0; r < RT; ++r)
                if (i0 + r * kEpiGroups < n_mine) P.out[(size_t)tt[r] * H + hh[r] * kBlock + row] = __float2bfloat16_rn(acc[r]);
        }
        if (etid == 0) MOE_STAMP_ALWAYS(14);
    }

    // ------------------------------------------------------------------ teardown
    tc_fence_before();
    const int gave_up = __syncthreads_or(wt.dead ? 1 : 0);
    tc_fence_after();
    // A launch in which some thread of this CTA gave up: nothing asynchronous may outlive the CTA.  Whatever each role
    // had requested -- weight and activation tiles by bulk copy, MMAs -- is waited for here (bounded), whether or not
    // the role itself noticed the give-up, before tensor memory is freed and shared memory goes to the next CTA.  (If no
    // thread of the CTA gave up, every role ran to its end: every tile requested was consumed, every MMA read back.)
    if (gave_up) {
        if (lane == 0 && (warp == 0 || warp == 2)) {
            const int cur = (int)misc[6 + (warp >> 1)];
            const uint32_t bar0 = warp ? bar_fullb : bar_full;
            for (int it = (cur > S ? cur - S : 0); it < cur; ++it)
                for (int i = 0; i < (1 << 20) && !mbar_try_wait(bar0 + 8 * (it % S), (uint32_t)((it / S) & 1)); ++i) {}
        }
        if (lane == 0 && (warp == 1 || warp == 3)) {
            const uint32_t bar = bar_drain + 8 * (uint32_t)(warp >> 1) * 2;
            umma_commit(bar);
            for (int i = 0; i < (1 << 20) && !mbar_try_wait(bar, 0); ++i) {}
        }
        tc_fence_before();
        __syncthreads();
        tc_fence_after();
    }
    if (warp == 1) tmem_dealloc(tmem_base, kTmemCols);
    if (tid == 0) {
        MOE_STAMP_ALWAYS(15);
        // Open the next epoch.  CTA 0 alone does it, without counting exits: it got here only after the grid-wide routing
        // wait, that is after every CTA had read this launch's tag; the next launch reads the epoch only once this grid
        // has completed.  (A fence and a returning atomic per CTA used to sit here: two L2 round trips at every exit.)
        // Unconditionally: a launch that gave up must not leave its tag to the next one.
        if (cta == 0) st_release(P.ctrl + kEpoch, tag);
    }
}

}  // namespace moe
