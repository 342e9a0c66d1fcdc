// Fused-unit variant of the routed-MoE decode kernel for 1..16 tokens (sm_100a).
//
// Same operator as moe_kernel.cuh (Section 3 of the paper: top-k/quantise, up projection, down projection, reduce, in
// one launch), laid out for the few-token case where the step is a chain of latencies rather than a stream:
//
//   * Work unit = (active expert e, 128-wide block ib of the intermediate dimension).  A unit is the gate and up rows
//     of that block over all of H (2 * H/128 weight tiles) FOLLOWED BY the down-projection column block
//     W2[e][:, 128 ib : 128 ib + 128] (H/128 tiles).  The intermediate block never leaves the chip: whoever finished
//     it streams the matching W2 tiles straight away and emits a partial down result per (token, slot, ib); the final
//     reduction sums top_k * I/128 partials per output element in fixed order.  No up->down flag, no intermediate
//     tile in global memory (Section 3.2 hands the tile over through a readiness flag; here the hand-over is local).
//   * A unit is shared by the C CTAs of a thread-block cluster (C = 1, 2, 4): rank r takes a contiguous part of the
//     H/128 K blocks of the gate/up rows and a contiguous part of the H/128 row blocks of the W2 column block.
//     Partial gate/up sums are exchanged through distributed shared memory (each CTA keeps its partial in its own
//     shared memory, peers read it with ld.shared::cluster after a remote mbarrier arrival) and every CTA of the
//     cluster computes the same SiLU(gate)*up, amax and FP8 codes (Section 3.3, up-projection epilogue) -- so the
//     intermediate tile needs no broadcast.  Launches in pairs decide after routing, from the number of units the
//     step really has, whether the CTAs of a pair share units or work alone.
//   * Units go to clusters whole, round-robin, or -- where a step has more units than clusters -- the list of all
//     accumulation groups is cut into equal ranges that may begin and end inside a unit; clusters that share a unit
//     exchange partial sums as tagged words.  Inside a cluster the stream is software-pipelined by one unit
//     (up(0) up(1) down(0) up(2) down(1) ...), so the exchange of unit i hides under the gate/up tiles of unit i+1.
//   * Router (Section 3.3): CTA c computes the logits of experts c, c+G, ... for all tokens with plain FMAs (the
//     rows were prefetched into L2 before the wait on the previous launch) and publishes each as one 64-bit word
//     {launch tag, logit}; every CTA polls those words directly -- one store trip plus one load trip, no counter,
//     no fence -- and selects for all tokens itself.  The down partials reach the final reduction the same way.
//   * Input quantisation (Section 4.1) is spread over the grid into the workspace and consumed by bulk-tensor copies,
//     behind an arrival counter that is off the critical path (the first activation tile is needed a first-tile
//     latency after the first weight request).
//   * One CTA per SM with a stage ring as deep as shared memory allows (two CTAs per SM with half the ring were
//     measured: the launch-to-launch interval does not shrink, the stream gets slower); the launch is made with the
//     programmatic-stream-serialization attribute, so the next launch's set-up and the L2 prefetch of its router rows
//     run ahead of its dependency wait.
//
// Warps: 0 producer (weight and activation tiles by bulk-tensor copy), 1..3 tcgen05 MMA issuers (take accumulation
// groups in turn, each with its own tensor-memory buffer), 4..7 accumulator/epilogue (thread = weight row), 8
// housekeeping during the routing phase (publishing and awaiting the quantised input, tensor-memory allocation).
#pragma once

#include "moe_kernel.cuh"

namespace moe {

constexpr int kFusedN = 16;                                   // MMA N of the fused variants (token t is column t)
constexpr int kFusedStage = kATileBytes + kFusedN * kBlock;    // weight tile + activation tile
constexpr int kFusedTmemBufs = 4;                              // accumulator buffers of 2 x 16 columns, one per MMA issuer
constexpr int kFusedIssuers = 3;                               // warps 1..3
constexpr int kFusedTmemCols = 128;
constexpr int kFusedThreads = 288;                             // 9 warps
// Wait-time accounting of the roles (cycle counts written next to the time stamps): compiled in only with
// -DMOE_FUSED_ACCOUNTING; reading the clock around every wait is not free on the short steps.
#ifdef MOE_FUSED_ACCOUNTING
#define MOE_CLK() clock64()
#else
#define MOE_CLK() 0ll
#endif
constexpr int kFusedMaxTok = 16;           // token columns of the widest instantiation (= MMA N)
constexpr int kFusedMaxRows = 4;          // router rows per CTA: ceil(kMaxExperts / 128)

// ---------------------------------------------------------------------------------------------
// cluster / distributed-shared-memory wrappers
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t cluster_ctarank() { uint32_t r; asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r)); return r; }
__device__ __forceinline__ uint32_t cluster_id_x() { uint32_t r; asm volatile("mov.u32 %0, %%clusterid.x;" : "=r"(r)); return r; }
__device__ __forceinline__ uint32_t cluster_nctarank() { uint32_t r; asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r)); return r; }
__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
__device__ __forceinline__ uint32_t map_to_rank(uint32_t saddr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
    return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t remote_bar) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(remote_bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait_cluster(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ float ld_cluster_f32(uint32_t addr) {
    float v;
    asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(addr) : "memory");
    return v;
}
// named barriers over a subset of the CTA's warps
__device__ __forceinline__ void named_bar_sync(int id, int nthreads) { asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory"); }
__device__ __forceinline__ void named_bar_arrive(int id, int nthreads) { asm volatile("bar.arrive %0, %1;" ::"r"(id), "r"(nthreads) : "memory"); }
__device__ __forceinline__ bool named_bar_and(int id, int nthreads, bool ok) {
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 p, %1, 0;\n\t"
        "bar.red.and.pred q, %2, %3, p;\n\t"
        "selp.u32 %0, 1, 0, q;\n\t}"
        : "=r"(r) : "r"((uint32_t)ok), "r"(id), "r"(nthreads) : "memory");
    return r != 0;
}
__device__ __forceinline__ unsigned long long ld_relaxed_u64(const unsigned long long* p) {
    unsigned long long v;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_relaxed_u64(unsigned long long* p, unsigned long long v) {
    asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}

// ---------------------------------------------------------------------------------------------
// shared-memory layout of the fused variants
// ---------------------------------------------------------------------------------------------
struct FusedSmem {
    int ring_off, hq_off, part_off, bar_off, misc_off, ids_off, w_off, mask_off, act_off, uidx_off, xs_off, red_off, poff_off, pair_off, total;
};
__host__ __device__ inline FusedSmem fused_smem_layout(int TC, int T, int K, int E, int H, int stages) {
    FusedSmem L;
    int o = 0;
    L.ring_off = o; o += stages * kFusedStage;                 // also the routing scratch (keys and score values) before the stream starts
    L.hq_off = o;   o += 2 * kFusedN * kBlock;                 // intermediate FP8 tile of the unit in flight, double-buffered (1024-byte aligned)
    L.part_off = o; o += 2 * 2 * TC * kBlock * 4;              // this CTA's partial gate/up sums [slot][gate TC | up TC][128 rows]; later the reduction scratch
    L.bar_off = o;  o += (2 * kMaxStages + 2 * kFusedTmemBufs + 12) * 8;
    L.misc_off = o; o += 64;
    L.ids_off = o;  o += T * K * 4;
    L.w_off = o;    o += T * K * 4;
    o = (o + 7) & ~7;
    L.mask_off = o; o += E * 16;
    L.act_off = o;  o += (E + 1) * 4;
    L.uidx_off = o; o += E * 4;
    o = (o + 15) & ~15;
    L.xs_off = o;   o += ((T + 3) & ~3) * (H / kBlock) * 4;    // input activation scales [H/128][T rounded up to 4]
    L.red_off = o;  o += 8 * kFusedMaxRows * kFusedMaxTok * 4;  // router partial dot products [warp][row][token]; later the amax scratch
    L.poff_off = o; o += E * 4;
    L.pair_off = o; o += ((T * K * 2 + 15) & ~15);
    L.total = o;
    return L;
}

// ---------------------------------------------------------------------------------------------
// the kernel.  TC = token columns the accumulator warps read (1, 2, 4, 8, 16 >= T).  SPLIT = the step may have more units
// than clusters, so the code that shares a unit between two clusters is compiled in (the host knows the largest unit
// count a token count can give; the instantiations without it are smaller and measurably faster on the short steps).
// Warps: 0 producer (weight and activation tiles), 1..3 MMA issuers, 4..7 accumulator warps; warp 8 keeps house
// during the routing phase (everything that costs L2 round trips but is not needed before the first activation tile).
// ---------------------------------------------------------------------------------------------
#ifndef MOE_FUSED_MIN_BLOCKS
#define MOE_FUSED_MIN_BLOCKS 1
#endif
template <int TC, bool SPLIT>
__global__ void __launch_bounds__(kFusedThreads, MOE_FUSED_MIN_BLOCKS)
moe_fused_kernel(const __grid_constant__ CUtensorMap tmW13, const __grid_constant__ CUtensorMap tmW2,
                 const __grid_constant__ CUtensorMap tmXq, const __grid_constant__ Params P) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);

    constexpr int N = kFusedN;
    constexpr int kMain = 256, kMainWarps = 8, kEpiThreads = 128;     // warps 0..7 share the routing phase; warp 8 keeps house meanwhile
    constexpr int kBufs = kFusedTmemBufs, kBufCols = 2 * N;          // an accumulator buffer = two 16-column halves
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int cta = blockIdx.x, G = gridDim.x;
    // LC = the cluster size of the launch.  C, nCl, rank, cl = how the CTAs work: as the launch says or -- decided after
    // routing, see there -- every CTA on its own although launched in pairs.
    const int LC = P.fC;
    int C = LC, nCl = P.fnCl, rank = (int)cluster_ctarank(), cl = (int)cluster_id_x();
    unsigned long long gmagic = P.grid_magic;                     // division by the number of (working) clusters
    const int T = (TC == 1) ? 1 : P.T;                          // (one token column means one token: its loops fold)
    const int H = P.H, E = P.E, I = P.I, K = P.K;
    const int KBu = H / kBlock, IB = I / kBlock, HB = H / kBlock;
    const int S = P.stages;
    const FusedSmem L = fused_smem_layout(TC, T, K, E, H, S);
    const int TS = (T + 3) & ~3;

    uint64_t* bars = (uint64_t*)(smem + L.bar_off);
    const uint32_t bar_full = smem_u32(bars), bar_empty = smem_u32(bars + kMaxStages);
    const uint32_t bar_tfull = smem_u32(bars + 2 * kMaxStages), bar_tempty = smem_u32(bars + 2 * kMaxStages + kBufs);
    const uint32_t bar_x = smem_u32(bars + 2 * kMaxStages + 2 * kBufs);
    const uint32_t bar_hq = bar_x, bar_xfull = bar_x + 16, bar_xfree = bar_x + 32, bar_drain = bar_x + 48, bar_hk = bar_x + 80;   // 2 + 2 + 2 + 4 + 1
    uint32_t* misc = (uint32_t*)(smem + L.misc_off);   // [0] tmem base, [1] U, [3] accumulator give-up, [5] ticket for reduction tasks, [6] quantised input published (1) or given up (2)
    int* s_ids = (int*)(smem + L.ids_off);
    float* s_w = (float*)(smem + L.w_off);
    unsigned long long* s_mask = (unsigned long long*)(smem + L.mask_off);
    int* s_act = (int*)(smem + L.act_off);
    float* s_xs = (float*)(smem + L.xs_off);
    float* s_red = (float*)(smem + L.red_off);
    int* s_poff = (int*)(smem + L.poff_off);
    unsigned short* s_pair = (unsigned short*)(smem + L.pair_off);
    float* s_part = (float*)(smem + L.part_off);
    uint8_t* s_hq = smem + L.hq_off;

    // ------------------------------------------------------------------ set-up ahead of the previous launch's end
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (warp == 0 && lane == 0) {
        tma_prefetch_desc(&tmW13); tma_prefetch_desc(&tmW2); tma_prefetch_desc(&tmXq);
        for (int s = 0; s < S; ++s) { mbar_init(bar_full + 8 * s, 1); mbar_init(bar_empty + 8 * s, 1); }
        for (int b = 0; b < kBufs; ++b) { mbar_init(bar_tfull + 8 * b, 1); mbar_init(bar_tempty + 8 * b, 4); }
        for (int b = 0; b < 2; ++b) {
            mbar_init(bar_hq + 8 * b, 1);
            mbar_init(bar_xfull + 8 * b, 4 * LC);             // one arrival per accumulator warp of every CTA of the cluster
            mbar_init(bar_xfree + 8 * b, 4 * LC);
        }
        for (int b = 0; b < 4; ++b) mbar_init(bar_drain + 8 * b, 1);
        mbar_init(bar_hk, 1);
        misc[3] = 0u; misc[5] = 0xFFFFFFFFu; misc[6] = 0u; misc[7] = 0u;
        fence_barrier_init();
    }
    if (warp == kMainWarps) { tmem_alloc(smem_u32(misc), kFusedTmemCols); tmem_relinquish(); }
#pragma unroll 1
    for (int e = tid; e < 2 * E; e += kFusedThreads) s_mask[e] = 0ull;
    // This CTA's router rows: ask L2 for them now.  (Weights are not written by the previous launch, and a prefetch
    // reads nothing into the SM.)
#pragma unroll 1
    for (int e = cta; e < E; e += G)
        for (int l = tid; l < H / 64; l += kFusedThreads) prefetch_l2(reinterpret_cast<const char*>(P.Wr + (size_t)e * H) + l * 128);
    if (P.bias && tid * 32 < E) prefetch_l2(P.bias + tid * 32);
    // Every CTA of the cluster must have initialised its barriers before anyone arrives on them remotely.  Real
    // clusters wait for that here (measured: starting the CTAs of a cluster in step is worth more than the wait costs);
    // a cluster of one only has to pair the arrival with a wait somewhere before the barrier's second use.
    cluster_arrive();
    const bool late_wait = (LC == 1) || ((P.fdyn & 3) == 2);          // (pairs that are expected to work alone do not meet here either)
    if (!late_wait) cluster_wait();
    asm volatile("griddepcontrol.wait;" ::: "memory");

    Waiter wt;
    wt.init(P.ctrl, P.timeout_ns);
    // The launch tag.  A relaxed load: everything the previous launch wrote is visible after the wait above, and an
    // acquire here would hold back the loads of the router phase for an L2 round trip.
    unsigned tag;
    asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(tag) : "l"(P.ctrl + kEpoch) : "memory");
    tag += 1u;
    if (tid == 0) MOE_STAMP(0);
    __syncwarp();             // (a lone lane that took a stamp rejoins its warp here, not somewhere inside the next loop)

    // ------------------------------------------------------------------ router logits of this CTA's experts (Section 3.3)
    if (warp < kMainWarps) {
        const int chunks = H / 8;                                 // 16-byte chunks per row
        int nrows = 0;
#pragma unroll 1
        for (int e = cta; e < E; e += G, ++nrows) {
            float acc[TC];
#pragma unroll
            for (int t = 0; t < TC; ++t) acc[t] = 0.f;
            const uint4* wrow = reinterpret_cast<const uint4*>(P.Wr + (size_t)e * H);
#pragma unroll 2
            for (int c = tid; c < chunks; c += kMain) {
                const uint4 wv = __ldg(wrow + c);
                uint4 xv[TC];
#pragma unroll
                for (int t = 0; t < TC; ++t) xv[t] = (t < T) ? __ldg(reinterpret_cast<const uint4*>(P.hidden + (size_t)t * H) + c) : make_uint4(0u, 0u, 0u, 0u);
                const uint32_t ww[4] = {wv.x, wv.y, wv.z, wv.w};
#pragma unroll
                for (int t = 0; t < TC; ++t) {
                    const uint32_t xx[4] = {xv[t].x, xv[t].y, xv[t].z, xv[t].w};
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        acc[t] = fmaf(__uint_as_float(ww[j] << 16), __uint_as_float(xx[j] << 16), acc[t]);
                        acc[t] = fmaf(__uint_as_float(ww[j] & 0xFFFF0000u), __uint_as_float(xx[j] & 0xFFFF0000u), acc[t]);
                    }
                }
            }
#pragma unroll
            for (int t = 0; t < TC; ++t) {
#pragma unroll
                for (int o = 16; o; o >>= 1) acc[t] += __shfl_xor_sync(0xffffffffu, acc[t], o);
                if (lane == 0) s_red[(warp * kFusedMaxRows + nrows) * kFusedMaxTok + t] = acc[t];
            }
        }
        named_bar_sync(2, kMain);
        if (tid < nrows * TC) {
            const int r = tid / TC, t = tid - r * TC;
            if (t < T) {
                float v = 0.f;
#pragma unroll
                for (int w = 0; w < kMainWarps; ++w) v += s_red[(w * kFusedMaxRows + r) * kFusedMaxTok + t];
                st_relaxed_u64(P.ll + (size_t)t * E + cta + r * G, ((unsigned long long)tag << 32) | (unsigned long long)__float_as_uint(v));
            }
        }
        if (tid == 0) MOE_STAMP(1);
        __syncwarp();
        // -------------------------------------------------------------- input quantisation (Section 4.1), spread over the grid
        const int groups = T * KBu;
#pragma unroll 1
        for (int p = (G - 1 - cta) * kMainWarps + warp; p < groups; p += G * kMainWarps) {   // from the last CTA down: the first ones have router rows
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
        // generic writes of xq -> the async proxy (bulk-tensor copies) of every CTA.  By every warp, also those that wrote
        // nothing of xq: the fence pushes out the thread's stores in flight, the router logits just published among them
        // (measured: without it the step is 1-1.5 us longer -- the logits reach the other CTAs later).
        fence_proxy_async();
        named_bar_arrive(3, kFusedThreads);                     // hand over to the housekeeping warp, do not wait for it
    } else {
        // ---------------------------------------------------------- housekeeping warp: everything that costs L2 round
        // trips but is not needed before the first activation tile.  Publish this CTA's share of the quantised input
        // (the release waits for the CTA's stores), wait until every CTA has, fetch the input scales.
        const unsigned par = tag & 1u;
        if (cta == 0 && lane == 0) {      // counters of the other launch parity start from zero next time
            P.ctrl[kRouteCnt + (par ^ 1u)] = 0u; P.ctrl[kRouteCnt2 + (par ^ 1u)] = 0u;
            P.ctrl[kQuantCnt + (par ^ 1u)] = 0u; P.ctrl[kDoneCnt + (par ^ 1u)] = 0u;
        }
#pragma unroll 1
        for (int e = cta * 32 + lane; e < kMaxPasses * E; e += G * 32) P.e_cnt[(par ^ 1u) * kMaxPasses * E + e] = 0u;
        named_bar_sync(3, kFusedThreads);
        bool okq = true;
        if (lane == 0) {
            red_release_add(P.ctrl + kQuantCnt + par, 1u);
            MOE_STAMP(2);
            okq = wt.flag(P.ctrl + kQuantCnt + par, (unsigned)G, 22);
        }
        okq = __shfl_sync(0xffffffffu, okq, 0);
        if (okq) {
#pragma unroll 1
            for (int i = lane; i < T * KBu; i += 32) { const int tt = div_small(i, KBu); s_xs[(i - tt * KBu) * TS + tt] = __ldcg(P.xs + i); }
        }
        fence_proxy_async();                 // what the counter's acquire made visible -> the producer's bulk-tensor reads of xq
        __syncwarp();
        if (lane == 0 && okq) mbar_arrive(bar_hk);      // the quantised input and its scales are there (never, if the wait gave up)
    }
    const uint32_t tmem_base = misc[0];

    // ------------------------------------------------------------------ gather all logits: poll the tagged words themselves
    uint32_t* s_key = reinterpret_cast<uint32_t*>(smem);
    float* s_val = reinterpret_cast<float*>(smem) + T * E;
    bool alive = true;
    if (warp < kMainWarps) {
        const bool softmax = (P.scoring == 0);
        bool ok = true;
#pragma unroll 1
        for (int p0 = tid; p0 < T * E && ok; p0 += 8 * kMain) {              // eight words in flight per thread
            unsigned long long v[8];
            unsigned pending = 0u;
#pragma unroll
            for (int j = 0; j < 8; ++j) if (p0 + j * kMain < T * E) pending |= 1u << j;
            for (uint32_t it = 1; pending; ++it) {
#pragma unroll
                for (int j = 0; j < 8; ++j) if (pending & (1u << j)) v[j] = ld_relaxed_u64(P.ll + p0 + j * kMain);
#pragma unroll
                for (int j = 0; j < 8; ++j) if ((pending & (1u << j)) && (unsigned)(v[j] >> 32) == tag) pending &= ~(1u << j);
                if (pending && (it & 63u) == 0 && wt.expired(20)) { ok = false; break; }
            }
            if (!ok) break;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int p = p0 + j * kMain;
                if (p < T * E) {
                    const float l = __uint_as_float((unsigned)v[j]);
                    if (cta == 0) P.logits[p] = l;
                    if (softmax) {
                        s_val[p] = l;
                        s_key[p] = orderable(l);
                    } else {
                        const float sg = __fdiv_rn(1.0f, 1.0f + expf(-l));
                        const float b = P.bias ? __ldg(P.bias + (p - div_small(p, E) * E)) : 0.f;
                        s_val[p] = sg;
                        s_key[p] = orderable(sg + b);
                    }
                }
            }
        }
        alive = named_bar_and(2, kMain, ok && !wt.dead);
        if (P.stamps_fine) { if (tid == 0) MOE_STAMP(3); __syncwarp(); }
        // -------------------------------------------------------------- top-k for every token, in every CTA (Section 4.1)
        // Token t is selected by warp 7 - t: the accumulator warps come first (they have a first-tile latency to spare),
        // the producer and the issuers last.  Only the ids and the token masks are needed to start the weight stream;
        // the routing weights are computed after the barrier.
        // (more than eight tokens: a second round; a warp then keeps two selections until the weights are computed)
        constexpr int kRounds = (TC + kMainWarps - 1) / kMainWarps;
        int my_id[kRounds];
        float my_v[kRounds], my_total[kRounds];
#pragma unroll
        for (int r = 0; r < kRounds; ++r) {
            my_id[r] = 0; my_v[r] = 0.f; my_total[r] = 1.f;
            const int my_t = r * kMainWarps + kMainWarps - 1 - warp;
            if (alive && my_t < T) {
                if (E <= 128) my_id[r] = route_pick<4>(P, my_t, lane, s_key + my_t * E, s_ids, s_mask);
                else if (E <= 256) my_id[r] = route_pick<8>(P, my_t, lane, s_key + my_t * E, s_ids, s_mask);
                else my_id[r] = route_pick<16>(P, my_t, lane, s_key + my_t * E, s_ids, s_mask);
                my_v[r] = route_vals(P, lane, my_id[r], s_val + my_t * E, my_total[r]);     // (the score table lies in the stage ring: read before the stream may start)
            }
        }
        named_bar_sync(2, kMain);            // the selected experts and token masks of every token are in shared memory
        if (P.stamps_fine) { if (tid == 0) MOE_STAMP(4); __syncwarp(); }
#pragma unroll
        for (int r = 0; r < kRounds; ++r) {
            const int my_t = r * kMainWarps + kMainWarps - 1 - warp;
            if (alive && my_t < T) route_weights(P, my_t, lane, my_id[r], my_v[r], my_total[r], s_ids, s_w, cta == 0);
        }
    } else {
        alive = false;                       // (the housekeeping warp takes no further part)
    }
    // Routing metadata without another CTA-wide barrier: every warp that needs the list of active experts (ascending)
    // builds it itself -- a ballot per 32 experts; all of them write the same values -- and the accumulator warps build
    // the table of routed (token, slot) pairs among themselves.
    int U = 0;
    if (alive) {
#pragma unroll 1
        for (int e0 = 0; e0 < E; e0 += 32) {
            const int e = e0 + lane;
            const bool on = (e < E) && (s_mask[2 * e] != 0ull);
            const unsigned bsel = __ballot_sync(0xffffffffu, on);
            if (on) s_act[U + __popc(bsel & ((1u << lane) - 1u))] = e;
            U += __popc(bsel);
        }
        __syncwarp();
        if (warp >= kEpiWarp0) {
            // (token, slot) pairs grouped by expert, tokens ascending: entry r of expert e = its r-th token and the slot e holds for it
            const int etid = tid - kEpiWarp0 * 32;
            if (warp == kEpiWarp0) {
                int base = 0;
#pragma unroll 1
                for (int e0 = 0; e0 < E; e0 += 32) {
                    const int c = (e0 + lane < E) ? __popcll(s_mask[2 * (e0 + lane)]) : 0;
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
                s_pair[s_poff[ex] + __popcll(s_mask[2 * ex] & ((1ull << t) - 1ull))] = (unsigned short)(t | ((pi - t * K) << 8));
            }
            epi_bar(kEpiThreads);
        }
    }
    if (P.stamps_fine) { if (tid == 0) MOE_STAMP(5); __syncwarp(); }
    const int nU = U * IB;                                       // units of this step
    // this CTA's share of every unit: K blocks [kb_lo, kb_hi) of the gate/up rows, row blocks [hb_lo, hb_hi) of W2
    // Pairs or every CTA on its own?  A launch made with clusters of two where the host could not know (`fdyn`) decides
    // now that the step's units are counted: as many units as pairs or fewer -- every pair shares one (half of the K
    // blocks and half of the W2 row blocks each, sums exchanged over distributed shared memory); more -- every CTA
    // works alone on whole units or ranges, as if launched with clusters of one (the pairing then only places the two
    // CTAs next to each other).  The expected number of distinct experts says which it will usually be; routing that
    // crowds a few experts (8 tokens on the same 8 experts: 48 units instead of 312) gets the other arrangement
    // instead of leaving two thirds of the SMs without a unit.
    // (Long units -- 60 groups and more, the layers with 5120 and more hidden columns -- stay in pairs up to 80 % as many
    // units as CTAs and cut the group list into one range per pair instead: alone, every fifth CTA or more would be
    // without a unit while the others each stream megabytes.  Measured on the two TP8 shards at 6 and 8 tokens: 4-8 %.)
    const bool solo = (P.fdyn != 0) && (nU > nCl) && !((P.fdyn & 4) != 0 && nU * 5 <= G * 4);
    if (solo) { C = 1; nCl = G; rank = 0; cl = cta; gmagic = P.grid_magic1; }
    const int kb_lo = solo ? 0 : P.fkb[rank], kb_hi = solo ? KBu : P.fkb[rank + 1], nk = kb_hi - kb_lo;
    const int hb_lo = solo ? 0 : P.fhb[rank], hb_hi = solo ? KBu : P.fhb[rank + 1], nh = hb_hi - hb_lo;
    const int ngd = (nh + 1) >> 1;                               // down groups per unit
    // Which units this cluster works on.  Either whole units, dealt round-robin, or -- where the host allows it and the
    // step has more units than clusters (or the host asks for it regardless: few crowded experts leave most clusters
    // without a unit) -- the list of all groups, per unit nk gate/up groups followed by ngd down groups, is cut into
    // equal contiguous ranges, one per cluster (Section 3.2 gives each expert a group of CTAs; here a range may begin and
    // end anywhere inside a unit, and be shorter than a unit).  A cluster's range covers the units ua..ue, the first
    // from position xa and the last up to position xe of their Wg groups.  In the order the cluster works on them:
    //   HEAD piece  unit ue, groups [0, xe)   if the range ends inside a unit other than its first: exports, never imports
    //   whole units
    //   TAIL piece  unit ua, groups [xa, ..)  if the range starts inside a unit (or lies inside a single one)
    // A piece with gate/up groups whose cluster does not hold all of the unit's down groups EXPORTS its partial sums as
    // tagged words right after those groups; a piece with down groups that lacks some of the unit's gate/up groups
    // IMPORTS the partial sums of every other cluster that has some, and adds all of them in cluster order (so every
    // cluster that makes the unit's intermediate tile makes the same one).  Exports happen before anything the cluster
    // imports (head piece first, tail piece last; inside a piece the export precedes the import), and a cluster imports
    // only from clusters below it: nobody waits in a circle, and nobody's export waits for an import.
    const int Wg = nk + ngd, total_g = nU * Wg;
    const bool split = SPLIT && (P.fsplit != 0) && (nU > nCl || P.fsplit == 2);
    auto cut = [&](int c) -> int { return (c >= nCl) ? total_g : (int)div_grid((unsigned)c * (unsigned)total_g, gmagic); };
    int n, first_whole = 0, nw = 0, hs = 0, ua = 0, xa = 0, ue = 0, xe = 0;
    bool has_tail = false;
    if (split) {
        const int lo = cut(cl), hi = cut(cl + 1);
        n = 0;
        if (hi > lo) {
            ua = lo / Wg; xa = lo - ua * Wg;
            ue = (hi - 1) / Wg; xe = hi - ue * Wg;                       // 0 < xe <= Wg
            hs = (ue > ua && xe < Wg) ? 1 : 0;
            has_tail = (xa > 0) || (ua == ue && xe < Wg);
            first_whole = ua + (xa > 0 ? 1 : 0);
            nw = ((xe < Wg) ? ue - 1 : ue) - first_whole + 1;
            if (nw < 0) nw = 0;
            n = hs + nw + (has_tail ? 1 : 0);
        }
    } else {
        n = (cl < nU) ? (int)div_grid((unsigned)(nU - cl + nCl - 1), gmagic) : 0;   // units cl, cl + nCl, ... (grid_magic divides by the cluster count)
    }
    // item s of this cluster, in working order: unit u = (expert e, intermediate block ib), gate/up groups [g0, g1) of
    // this CTA's K blocks, down groups [d0, d1) of this CTA's row blocks (none: the item ends with its partial sums),
    // and whether its partial sums are exported and/or other clusters' imported
    constexpr int kExport = 1, kImport = 2;
    auto item_of = [&](int s, int& u, int& e, int& ib, int& g0, int& g1, int& d0, int& d1) -> int {
        int fl = 0;
        g0 = 0; g1 = nk; d0 = 0; d1 = ngd;
        if (!SPLIT || !split) u = cl + s * nCl;
        else {
            int x0 = 0, x1 = Wg;
            if (s < hs) { u = ue; x1 = xe; }
            else if (s - hs < nw) u = first_whole + s - hs;
            else { u = ua; x0 = xa; x1 = (ua == ue) ? xe : Wg; }
            g0 = x0 < nk ? x0 : nk; g1 = x1 < nk ? x1 : nk;
            d0 = x0 > nk ? x0 - nk : 0; d1 = x1 > nk ? x1 - nk : 0;
            if (g1 > g0 && !(d0 == 0 && d1 == ngd)) fl |= kExport;           // somebody else has down groups of this unit
            if (d1 > d0 && !(g0 == 0 && g1 == nk)) fl |= kImport;            // somebody else has gate/up groups of it
        }
        const int a = div_small(u, IB);
        ib = u - a * IB;
        e = s_act[a];
        return fl;
    };
    int Ntot = 0;                                                // weight tiles of this CTA
    for (int s = 0; s < n; ++s) {
        int u, e, ib, g0, g1, d0, d1;
        item_of(s, u, e, ib, g0, g1, d0, d1);
        Ntot += 2 * (g1 - g0) + ((2 * d1 < nh ? 2 * d1 : nh) - 2 * d0);     // (a unit's last down group may be a single tile)
    }

    // Stream order of this CTA (same in every role): for s = 0..n: the gate/up groups of unit s (if s < n), then the
    // down groups of unit s-1 (if s >= 1).  A group is what one accumulator buffer holds: two weight tiles -- the gate
    // and the up tile of one K block (columns [0,16) and [16,32), activation tile next to the gate tile), or two
    // consecutive row blocks of the W2 column block (activation operand = the on-chip intermediate tile) -- or a
    // single last W2 tile.  One mbarrier per group in each direction: the group's tiles land on the `full` barrier of
    // its first stage and are released through that stage's `empty` barrier, so a stage that was the second of a pair
    // needs no wait of its own (the ring is refilled in order: its pair-mate's release came first).
    const int NI = (S >> 1) < kFusedIssuers ? (S >> 1) : kFusedIssuers;   // MMA issuers = accumulator buffers in use
    // ------------------------------------------------------------------ role: producer (weight tiles and activation tiles)
    if (warp == 0) {
        if (lane == 0 && alive && n > 0) {
            const uint64_t stream_once = l2_policy_evict_first();
            wt.mbar(bar_hk, 0u, 22);             // the quantised input of every CTA is published and fenced for bulk copies (housekeeping warp); long done by now
            int cur = 0, st = 0;
            long long w_empty = 0;
            uint32_t cntpar = 0u, second = 0u;   // per stage: parity of the number of groups it anchored; last filled as the second tile of a pair
            // one group: 1 or 2 weight tiles (rows y0 / y1 of `m`, column x) and, for gate/up groups, the activation tile of K block xq_kb
            auto put = [&](const CUtensorMap* m, int x0, int y0, int x1, int y1, int ntiles, int xq_kb) -> bool {
                const int st0 = st, st1 = (st + 1 == S) ? 0 : st + 1;
                const long long c0 = MOE_CLK();
                if (!((second >> st0) & 1u) && !wt.mbar(bar_empty + 8 * st0, ((cntpar >> st0) & 1u) ^ 1u, 21)) return false;
                if (ntiles == 2 && !((second >> st1) & 1u) && !wt.mbar(bar_empty + 8 * st1, ((cntpar >> st1) & 1u) ^ 1u, 21)) return false;
                w_empty += MOE_CLK() - c0;
                const uint32_t full = bar_full + 8 * st0, dst0 = smem_u32(smem) + (uint32_t)st0 * kFusedStage;
                mbar_expect_tx(full, (uint32_t)(ntiles * kATileBytes + (xq_kb >= 0 ? N * kBlock : 0)));
                tma_load_2d_hint(dst0, m, x0, y0, full, stream_once);
                if (xq_kb >= 0) tma_load_2d(dst0 + kATileBytes, &tmXq, xq_kb * kBlock, 0, full);   // rows 0..15 of xq (tokens beyond T are never read back)
                if (ntiles == 2) tma_load_2d_hint(smem_u32(smem) + (uint32_t)st1 * kFusedStage, m, x1, y1, full, stream_once);
                cntpar ^= 1u << st0;
                second &= ~(1u << st0);
                if (ntiles == 2) second |= 1u << st1;
                cur += ntiles;
                st += ntiles; if (st >= S) st -= S;
                return true;
            };
            MOE_STAMP(6);
            for (int s = 0; s <= n && !wt.dead; ++s) {
                if (s < n) {
                    int u, e, ib, g0, g1, d0, d1;
                    item_of(s, u, e, ib, g0, g1, d0, d1);
                    const int yg = e * 2 * I + ib * kBlock;
                    for (int k = kb_lo + g0; k < kb_lo + g1; ++k)
                        if (!put(&tmW13, k * kBlock, yg, k * kBlock, yg + I, 2, k)) break;
                }
                if (s >= 1 && !wt.dead) {
                    int u, e, ib, g0, g1, d0, d1;
                    item_of(s - 1, u, e, ib, g0, g1, d0, d1);
                    for (int h = hb_lo + 2 * d0; h < hb_hi && h < hb_lo + 2 * d1; h += 2)
                        if (!put(&tmW2, ib * kBlock, e * H + h * kBlock, ib * kBlock, e * H + (h + 1) * kBlock, (h + 1 < hb_hi) ? 2 : 1, -1)) break;
                }
            }
            if (P.stamps) P.stamps[(size_t)blockIdx.x * kStampsPerCta + 16] = (unsigned long long)w_empty;
            misc[7] = cntpar;      // which phase of every stage's `full` barrier was armed last (the teardown waits for them if the launch gave up)
        }
        // Every copy of this CTA is requested (or it has no unit at all): take a ticket for a share of the final
        // reduction now, so that it is there when the CTA gets to it.  Tickets go out in the order in which CTAs run out
        // of work: the reduction is done by those that finish early, and the last CTA to finish finds none left.
        if (SPLIT && lane == 0 && alive && !wt.dead) misc[5] = atomicAdd(P.ctrl + kDoneCnt + (tag & 1u), 1u);
        __syncwarp();
    }
    // ------------------------------------------------------------------ role: MMA issuers
    // Measured in this kernel: one group (two waits, a fence, eight tcgen05.mma, two commits) occupies its issuing thread
    // for about 1100 cycles, far longer than the tensor pipe needs for it.  So three threads (warps 1, 2, 3)
    // take the groups in turn, each with the accumulator buffer of its own number; all of them walk the whole sequence
    // to keep the stage positions and barrier phases.  Commits are kept few -- one `empty` and one `full` per group,
    // no `empty` for stages that are never refilled.  With NI issuers and NI buffers nobody runs more than NI groups
    // ahead of the slowest (a buffer is handed back only after every earlier group was read), and NI <= S/2 groups is
    // less than a lap of the ring: a parity wait on a stage can never be a phase off.
    else if (warp < kEpiWarp0) {
        const int iss = warp - 1;
        if (lane == 0 && alive && n > 0 && iss < NI) {
            constexpr uint32_t idesc = (1u << 4) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(kBlock >> 4) << 24);
            const uint32_t ring = smem_u32(smem);
            int st = 0, j = 0, turn = 0;
            uint32_t fpar = 0u;                  // per stage: parity of the next phase of its `full` barrier
            uint32_t tpar = 1u;                  // parity to wait for on this issuer's `tempty` barrier
            long long w_te = 0, w_fu = 0, w_hq = 0, w_is = 0;
            bool first = true;
            // one group: tile(s) at stage st (and st + 1), activation operand at b_addr (0: next to the first tile)
            auto group = [&](int ntiles, uint32_t b_addr) -> bool {
                const int st0 = st, st1 = (st + 1 == S) ? 0 : st + 1;
                const bool mine = (turn == iss);
                const bool release = (j + S < Ntot);              // a later tile will take this stage
                st += ntiles; if (st >= S) st -= S;
                j += ntiles;
                if (++turn == NI) turn = 0;
                const uint32_t fp = (fpar >> st0) & 1u;
                fpar ^= 1u << st0;
                if (!mine) return true;
                const long long c0 = MOE_CLK();
                if (!wt.mbar(bar_tempty + 8 * iss, tpar, 24)) return false;
                tpar ^= 1u;
                const long long c1 = MOE_CLK();
                if (!wt.mbar(bar_full + 8 * st0, fp, 26)) return false;
                const long long c2 = MOE_CLK();
                w_te += c1 - c0; w_fu += c2 - c1;
                if (first && iss == 0) { MOE_STAMP(7); first = false; }
                const uint32_t a0 = ring + (uint32_t)st0 * (uint32_t)kFusedStage;
                const uint64_t b_desc = make_smem_desc(b_addr ? b_addr : a0 + kATileBytes);
                const uint32_t d = tmem_base + (uint32_t)(iss * kBufCols);
                tc_fence_after();
                {
                    const uint64_t a_desc = make_smem_desc(a0);
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk) umma_f8(d, a_desc + (uint64_t)(kk * 2), b_desc + (uint64_t)(kk * 2), idesc, kk > 0 ? 1u : 0u);
                }
                if (ntiles == 2) {
                    const uint64_t a_desc = make_smem_desc(ring + (uint32_t)st1 * (uint32_t)kFusedStage);
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk) umma_f8(d + N, a_desc + (uint64_t)(kk * 2), b_desc + (uint64_t)(kk * 2), idesc, kk > 0 ? 1u : 0u);
                }
                if (release) umma_commit(bar_empty + 8 * st0);
                umma_commit(bar_tfull + 8 * iss);
                w_is += MOE_CLK() - c2;
                return true;
            };
            int dq = 0;                                            // items with down groups so far: slot and phase of the intermediate tile
            for (int s = 0; s <= n && !wt.dead; ++s) {
                if (s < n) {
                    int u, e, ib, g0, g1, d0, d1;
                    item_of(s, u, e, ib, g0, g1, d0, d1);
                    for (int k = g0; k < g1; ++k)
                        if (!group(2, 0u)) break;
                }
                if (s >= 1 && !wt.dead) {
                    int u, e, ib, g0, g1, d0, d1;
                    item_of(s - 1, u, e, ib, g0, g1, d0, d1);
                    if (d1 <= d0) continue;                                  // (a head piece that ends with its partial sums)
                    const int slot = dq & 1;
                    // the intermediate tile of the item is in shared memory (written by the accumulator warps)
                    { const long long c0 = MOE_CLK(); if (!wt.mbar(bar_hq + 8 * slot, (uint32_t)((dq >> 1) & 1), 27)) break; w_hq += MOE_CLK() - c0; }
                    ++dq;
                    for (int h = 2 * d0; h < nh && h < 2 * d1; h += 2)
                        if (!group((h + 1 < nh) ? 2 : 1, smem_u32(s_hq) + (uint32_t)(slot * N * kBlock))) break;
                }
            }
            if (P.stamps && iss == 0) { unsigned long long* o = P.stamps + (size_t)blockIdx.x * kStampsPerCta; o[17] = w_te; o[18] = w_fu; o[19] = w_hq; o[20] = w_is; }
        }
        __syncwarp();
    }
    // ------------------------------------------------------------------ role: accumulator / epilogue warps
    else if (warp >= kEpiWarp0 && warp < kEpiWarp0 + 4) {
        if (late_wait) cluster_wait();                         // (pairs with the set-up's arrival)
        const int q = warp & 3, row = q * 32 + lane;           // TMEM lane == weight row inside the tile
        const int etid = tid - kEpiWarp0 * 32;
        const uint32_t t_lane = tmem_base + ((uint32_t)(q * 32) << 16);
        bool first_acc = true;
        float sc[TC];                                          // scale of the intermediate tile per token column (unit in its down phase)
#pragma unroll
        for (int c = 0; c < TC; ++c) sc[c] = 0.f;
        // wait for group g's accumulators, read the first TC columns of both halves of its buffer, hand the buffer back
        long long w_tf = 0, w_xf = 0, w_fc = 0;
        int buf = 0;
        uint32_t bpar = 0u;                                    // parity of the next phase of bar_tfull[buf]
        auto take = [&](float* d0, float* d1) {
            const long long c0 = MOE_CLK();
            if (!wt.mbar(bar_tfull + 8 * buf, bpar, 29)) misc[3] = 1u;
            w_tf += MOE_CLK() - c0;
            tc_fence_after();
            const uint32_t tcol = t_lane + (uint32_t)(buf * kBufCols);
            tmem_ld<TC>(tcol, d0);
            tmem_ld<TC>(tcol + N, d1);
            tmem_ld_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_tempty + 8 * buf);
            if (++buf == NI) { buf = 0; bpar ^= 1u; }
        };
        // Block scales of unit s for this CTA's tiles: lane l holds K block kb_lo + l (and + 32) of the gate and of the up
        // rows, and row block hb_lo + l (and + 32) of the W2 column block.  Fetched one unit ahead of their use.
        float nwg0 = 0.f, nwu0 = 0.f, nwg1 = 0.f, nwu1 = 0.f, nw2a = 0.f, nw2b = 0.f;
        auto fetch_scales = [&](int s) {
            if (s >= n) return;
            int u, e, ib, g0, g1, d0, d1;
            item_of(s, u, e, ib, g0, g1, d0, d1);
            const float* g13 = P.W13s + ((size_t)e * 2 * IB + ib) * KBu + kb_lo;
            const float* u13 = P.W13s + ((size_t)e * 2 * IB + IB + ib) * KBu + kb_lo;
            const float* w2 = P.W2s + ((size_t)e * HB + hb_lo) * IB + ib;
            nwg0 = (lane < nk) ? __ldg(g13 + lane) : 0.f;           nwu0 = (lane < nk) ? __ldg(u13 + lane) : 0.f;
            nwg1 = (lane + 32 < nk) ? __ldg(g13 + 32 + lane) : 0.f; nwu1 = (lane + 32 < nk) ? __ldg(u13 + 32 + lane) : 0.f;
            nw2a = (lane < nh) ? __ldg(w2 + (size_t)lane * IB) : 0.f;
            nw2b = (lane + 32 < nh) ? __ldg(w2 + (size_t)(lane + 32) * IB) : 0.f;
        };
        if (alive && n > 0) {
            fetch_scales(0);
            if (!wt.mbar(bar_hk, 0u, 28)) misc[3] = 1u;          // the input scales are in shared memory (housekeeping warp)
            float w2a = 0.f, w2b = 0.f, dw2a = 0.f, dw2b = 0.f;     // W2 scales of the unit in its gate/up phase, and of the one in its down phase
            unsigned dmask = 0u;                                   // token columns and result offsets of the unit in its down phase
            int dyoff = 0;
            bool d_valid = false;                                  // the previous item has down groups
            int dh0 = 0, dh1 = 0;                                  // ... for the row blocks [dh0, dh1) of this CTA's share
            int pk = 0, dq = 0;                                    // items parked for the cluster / items with an intermediate tile so far
            int pslot = 0;
            uint32_t pphase = 0u;
            for (int s = 0; s <= n; ++s) {
                int u = 0, e = 0, ib = 0, g0 = 0, g1 = 0, d0 = 0, d1 = 0, fl = 0;
                if (s < n) fl = item_of(s, u, e, ib, g0, g1, d0, d1);
                // ---------------- gate/up groups of item s: accumulate, then park the partial sums for the cluster
                if (s < n) {
                    const float wg0 = nwg0, wu0 = nwu0;
                    const float wg1 = nwg1, wu1 = nwu1;
                    w2a = nw2a; w2b = nw2b;
                    fetch_scales(s + 1);
                    float accg[TC], accu[TC];
#pragma unroll
                    for (int c = 0; c < TC; ++c) { accg[c] = 0.f; accu[c] = 0.f; }
#pragma unroll 1
                    for (int k = g0; k < g1; ++k) {
                        float dg[TC], du[TC];
                        take(dg, du);
                        if (first_acc) { if (etid == 0) MOE_STAMP(8); first_acc = false; }
                        const int kl = k & 31;
                        const float wsg = __shfl_sync(0xffffffffu, (k < 32) ? wg0 : wg1, kl), wsu = __shfl_sync(0xffffffffu, (k < 32) ? wu0 : wu1, kl);
                        const float* as = s_xs + (kb_lo + k) * TS;
#pragma unroll
                        for (int c = 0; c < TC; ++c) {
                            const float a = as[c];
                            accg[c] = fmaf(dg[c], wsg * a, accg[c]);
                            accu[c] = fmaf(du[c], wsu * a, accu[c]);
                        }
                    }
                    if (SPLIT && (fl & kExport)) {
                        // this CTA's partial sums go to the clusters that hold down groups of the unit, as tagged words (they add
                        // them at the very end of their ranges: they are there long before).  A cluster exports at most two
                        // pieces: the one of its first unit (slot 0) and the one of its last (slot 1).
                        unsigned long long* xo = P.xsl + ((size_t)((cl * 2 + (u == ua ? 0 : 1)) * C + rank) * 2 * TC) * kBlock + row;
                        const unsigned long long tagx = (unsigned long long)tag << 32;
                        const bool live = (misc[3] == 0u) && !wt.dead;
#pragma unroll
                        for (int c = 0; c < TC; ++c) {
                            if (live) {
                                st_relaxed_u64(xo + (size_t)c * kBlock, tagx | (unsigned long long)__float_as_uint(accg[c]));
                                st_relaxed_u64(xo + (size_t)(TC + c) * kBlock, tagx | (unsigned long long)__float_as_uint(accu[c]));
                            }
                        }
                    }
                    if (d1 > d0) {
                        // park: slot pk & 1 of this CTA's partial buffer, free once every peer has read the item that used it before
                        pslot = pk & 1; pphase = (uint32_t)((pk >> 1) & 1);
                        if (C > 1 && pk >= 2 && lane == 0) {
                            bool okw = !wt.dead;
                            for (uint32_t i = 1; okw && !mbar_try_wait_cluster(bar_xfree + 8 * pslot, pphase ^ 1u); ++i)
                                if ((i & 255u) == 0 && wt.expired(30)) okw = false;
                            if (!okw) misc[3] = 1u;
                        }
                        ++pk;
                        __syncwarp();
                        float* pp = s_part + pslot * 2 * TC * kBlock;
#pragma unroll
                        for (int c = 0; c < TC; ++c) { pp[c * kBlock + row] = accg[c]; pp[(TC + c) * kBlock + row] = accu[c]; }
                        __syncwarp();
                        if (C > 1 && lane < C) mbar_arrive_cluster(map_to_rank(bar_xfull + 8 * pslot, (uint32_t)lane));
                    }
                    if (s == 0 && etid == 0) MOE_STAMP(9);
                }
                // ---------------- two steps, normally in this order:
                //   down(s-1): the down groups of unit s-1 (its intermediate tile was made at the end of the previous turn, long
                //     before the issuers got here: no hand-over wait on the weight stream's path), scaled and stored as the
                //     tagged partials of (token, slot, ib): the final reduction polls these words themselves;
                //   F(s): gather the cluster's partial sums of unit s, SiLU*up, requantise -> the intermediate tile its down
                //     groups will use one turn later.
                // In the LAST turn with gate/up groups nothing follows that could hide F(s) -- the issuers go from the down
                // groups of s-1 straight to those of s -- so there F(s) comes first, while the down MMAs of s-1 run.
                const bool f_first = (s == n - 1);
                bool failed = false, n_valid = false;
                float nsc[TC];
                unsigned nmask = 0u;
                int nyoff = 0;
#pragma unroll
                for (int c = 0; c < TC; ++c) nsc[c] = 0.f;
#pragma unroll 1
                for (int step = 0; step < 2; ++step) {
                if ((step == 0) != f_first) {
                    if (s >= 1 && d_valid) {
                        const unsigned long long tagw = (unsigned long long)tag << 32;
#pragma unroll 1
                        for (int h = dh0; h < dh1; h += 2) {
                            float y0[TC], y1[TC];
                            take(y0, y1);
                            const float ws0 = __shfl_sync(0xffffffffu, (h < 32) ? dw2a : dw2b, h & 31);
                            const float ws1 = __shfl_sync(0xffffffffu, (h + 1 < 32) ? dw2a : dw2b, (h + 1) & 31);
                            unsigned long long* yrow = P.ypl + (size_t)(hb_lo + h) * kBlock + row;
                            const bool live = (misc[3] == 0u) && !wt.dead;     // never publish a result that was not computed
                            const bool two = (h + 1 < nh);
#pragma unroll
                            for (int c = 0; c < TC; ++c) {
                                const int yo = __shfl_sync(0xffffffffu, dyoff, c);
                                if (((dmask >> c) & 1u) && live) {
                                    st_relaxed_u64(yrow + (size_t)yo, tagw | (unsigned long long)__float_as_uint(y0[c] * (ws0 * sc[c])));
                                    if (two) st_relaxed_u64(yrow + (size_t)yo + kBlock, tagw | (unsigned long long)__float_as_uint(y1[c] * (ws1 * sc[c])));
                                }
                            }
                        }
                    }
                } else {
                    // ---------------- unit s: gather the cluster's partial sums, SiLU*up, requantise -> the intermediate tile its
                    // down groups will use one turn later
                    if (s < n && d1 > d0) {
                        const int slot = pslot;
                        // token columns of this expert and where their down results go
                        const unsigned mask = (unsigned)s_mask[2 * e];
                        int yoff_lane = 0;
                        if (lane < TC && ((mask >> lane) & 1u)) {
                            const unsigned pr = s_pair[s_poff[e] + __popc(mask & ((1u << lane) - 1u))];
                            yoff_lane = (((int)(pr & 0xFFu) * K + (int)(pr >> 8)) * IB + ib) * H;
                        }
                        const long long cf0 = MOE_CLK();
                        if (C > 1) {
                            bool okw = !wt.dead;
                            for (uint32_t it = 1; okw && !mbar_try_wait_cluster(bar_xfull + 8 * slot, pphase); ++it)
                                if ((it & 255u) == 0 && wt.expired(31)) okw = false;
                            if (!okw) misc[3] = 1u;
                        }
                        w_xf += MOE_CLK() - cf0;
                        float a[TC];
                        {
                            float sg[TC], su[TC];
#pragma unroll
                            for (int c = 0; c < TC; ++c) { sg[c] = 0.f; su[c] = 0.f; }
                            const uint32_t mine = smem_u32(s_part + slot * 2 * TC * kBlock) + (uint32_t)row * 4u;
                            if (C == 1) {
                                // a cluster of one: every thread reads back what it parked itself (no barrier, no cluster addressing)
                                const float* pp = s_part + slot * 2 * TC * kBlock + row;
#pragma unroll
                                for (int c = 0; c < TC; ++c) { sg[c] = 0.f + pp[c * kBlock]; su[c] = 0.f + pp[(TC + c) * kBlock]; }
                            }
#pragma unroll 1
                            for (int r = 0; r < C && C > 1; ++r) {             // rank order: every CTA of the cluster gets the same sums
                                const uint32_t src = map_to_rank(mine, (uint32_t)r);
                                float vg[TC], vu[TC];
#pragma unroll
                                for (int c = 0; c < TC; ++c) {                 // (columns of tokens not routed to this expert are dropped below)
                                    vg[c] = ld_cluster_f32(src + (uint32_t)(c * kBlock * 4));
                                    vu[c] = ld_cluster_f32(src + (uint32_t)((TC + c) * kBlock * 4));
                                }
#pragma unroll
                                for (int c = 0; c < TC; ++c) { sg[c] += vg[c]; su[c] += vu[c]; }
                            }
                            if (SPLIT && (fl & kImport)) {
                                // Other clusters worked on gate/up groups of this unit: the ones whose ranges meet the unit's gate/up
                                // positions [u Wg, u Wg + nk).  Their CTAs' partial sums are tagged words (polled, bounded; stored
                                // right after those groups, which every cluster works on before anything it imports for).
                                auto cluster_of = [&](int pos) -> int {
                                    int p = (int)(((unsigned)pos * (unsigned)nCl) / (unsigned)total_g);
                                    while (p + 1 < nCl && cut(p + 1) <= pos) ++p;
                                    while (p > 0 && cut(p) > pos) --p;
                                    return p;
                                };
                                const int p_lo = cluster_of(u * Wg), p_hi = cluster_of(u * Wg + nk - 1);
                                bool okx = !wt.dead;
#pragma unroll 1
                                for (int p = p_lo; p <= p_hi && okx; ++p) {
                                    if (p == cl || cut(p + 1) == cut(p)) continue;            // (a cluster with an empty range exports nothing)
                                    const int pslot_x = (cut(p) / Wg == u) ? 0 : 1;          // the unit is that cluster's first one, or its last
                                    const unsigned long long* xi = P.xsl + ((size_t)((p * 2 + pslot_x) * C) * 2 * TC) * kBlock + row;
#pragma unroll 1
                                    for (int r = 0; r < C && okx; ++r) {
                                        // all 2 TC words of a source at once up to eight columns; the gate columns, then the up
                                        // columns beyond (32 words in flight would cost 64 registers)
                                        constexpr int kPass = (TC > 8) ? 2 : 1, kW = 2 * TC / kPass;
#pragma unroll 1
                                        for (int pass = 0; pass < kPass && okx; ++pass) {
                                            unsigned long long v[kW];
                                            unsigned pending = (1u << kW) - 1u;
                                            for (uint32_t it = 1; pending; ++it) {
#pragma unroll
                                                for (int c = 0; c < kW; ++c) if (pending & (1u << c)) v[c] = ld_relaxed_u64(xi + ((size_t)r * 2 * TC + pass * kW + c) * kBlock);
#pragma unroll
                                                for (int c = 0; c < kW; ++c) if ((pending & (1u << c)) && (unsigned)(v[c] >> 32) == tag) pending &= ~(1u << c);
                                                if (pending && (it & 63u) == 0 && wt.expired(34)) { okx = false; break; }
                                            }
                                            if (!okx) break;
                                            if (kPass == 1) {
#pragma unroll
                                                for (int c = 0; c < TC; ++c) { sg[c] += __uint_as_float((unsigned)v[c]); su[c] += __uint_as_float((unsigned)v[(kW > TC ? TC : 0) + c]); }
                                            } else {
#pragma unroll
                                                for (int c = 0; c < TC; ++c) { if (pass == 0) sg[c] += __uint_as_float((unsigned)v[c]); else su[c] += __uint_as_float((unsigned)v[c]); }
                                            }
                                        }
                                    }
                                }
                                if (!okx) misc[3] = 1u;
                            }
                            // SiLU(gate)*up (Section 3.3).  The intermediate tile is outside the bit-exact set: fast exp and divide.
#pragma unroll
                            for (int c = 0; c < TC; ++c) a[c] = ((mask >> c) & 1u) ? __fdividef(sg[c], 1.0f + __expf(-sg[c])) * su[c] : 0.f;
                        }
                        __syncwarp();
                        if (C > 1 && lane < C) mbar_arrive_cluster(map_to_rank(bar_xfree + 8 * slot, (uint32_t)lane));   // my reads of every peer's slot are done
                        // 128-wide amax per token column: warp maximum (as an integer: |a| orders like its bits), then across the four warps
#pragma unroll
                        for (int c = 0; c < TC; ++c) {
                            const uint32_t m = __reduce_max_sync(0xffffffffu, __float_as_uint(fabsf(a[c])));
                            if (lane == 0) s_red[q * kFusedMaxTok + c] = __uint_as_float(m);
                        }
                        if (!epi_all(misc[3] == 0u && !wt.dead, kEpiThreads)) { wt.dead = true; failed = true; break; }
                        const int hslot = dq & 1;
                        ++dq;
                        uint8_t* hq = s_hq + hslot * N * kBlock;
#pragma unroll
                        for (int c = 0; c < TC; ++c) {
                            const float amax = fmaxf(fmaxf(s_red[c], s_red[kFusedMaxTok + c]), fmaxf(s_red[2 * kFusedMaxTok + c], s_red[3 * kFusedMaxTok + c]));
                            nsc[c] = fmaxf(amax, 1e-10f) * (1.0f / 448.0f);     // (the intermediate tile's scale is outside the bit-exact set)
                        }
#pragma unroll
                        for (int c = 0; c < TC; ++c) {
                            if ((mask >> c) & 1u) {
                                const float2 v = make_float2(a[c] * __fdividef(1.0f, nsc[c]), 0.f);
                                // K-major, 128-byte swizzled B tile: row = token column, 16-byte chunk (row >> 4) sits at chunk ^ (column & 7)
                                hq[c * kBlock + ((((row >> 4) ^ (c & 7)) << 4) | (row & 15))] = (uint8_t)(__nv_cvt_float2_to_fp8x2(v, __NV_SATFINITE, __NV_E4M3) & 0xFF);
                            }
                        }
                        fence_proxy_async_smem();                              // generic shared-memory writes -> the tensor core's reads (not the tagged global stores in flight)
                        epi_bar(kEpiThreads);
                        if (etid == 0) { if (!(P.debug_skip & 1)) mbar_arrive(bar_hq + 8 * hslot); if (dq == 1) MOE_STAMP(10); }
                        w_fc += MOE_CLK() - cf0;
                        nmask = mask; nyoff = yoff_lane; n_valid = true;
                    }
                }
                }
                if (failed) break;
                // unit s moves into its down phase
#pragma unroll
                for (int c = 0; c < TC; ++c) sc[c] = nsc[c];
                dmask = nmask; dyoff = nyoff; dw2a = w2a; dw2b = w2b; d_valid = n_valid;
                dh0 = 2 * d0; dh1 = (2 * d1 < nh) ? 2 * d1 : nh;
            }
        }
        if (etid == 0) { MOE_STAMP(11); if (P.stamps) { unsigned long long* o = P.stamps + (size_t)blockIdx.x * kStampsPerCta; o[21] = w_tf; o[22] = w_xf; o[23] = w_fc; } }
    }

    // ------------------------------------------------------------------ final weighted reduction (Section 3.2: only this
    // remains in the drain); deterministic.  Task = (token, 32 rows), task = (G - 1 - cta) + i * G, lane = row.  The top_k * I/128
    // (slot, ib) partials of a task are tagged words: a reader polls them until they carry this launch's tag -- their
    // producers' stores need no flag, no fence and no counter.  `sp` warps share a task (8 when a CTA has one task, 1
    // when it has eight or more), warp part q of them taking the partials q, q + sp, ...; their sums are combined in
    // fixed order.  sp depends only on the shape, the token count and the grid.
    tc_fence_before();
    const int gave_up = __syncthreads_or((wt.dead || misc[3] != 0u) ? 1 : 0);
    tc_fence_after();
    // A launch in which some thread of this CTA gave up: nothing asynchronous may outlive the CTA.  The bulk copies the
    // producer had requested and the MMAs the issuers had issued are waited for here (bounded), whether or not those
    // roles noticed the give-up themselves, before tensor memory is freed and shared memory goes to the next CTA.  (If
    // no thread of the CTA gave up, every role ran to its end: every tile requested was consumed, every MMA read back.)
    if (gave_up) {
        if (tid == 0) {
            const uint32_t cntpar = misc[7];
            for (int s = 0; s < S; ++s)
                for (int i = 0; i < (1 << 18) && !mbar_try_wait(bar_full + 8 * s, ((cntpar >> s) & 1u) ^ 1u); ++i) {}
        }
        if (lane == 0 && warp >= 1 && warp < kEpiWarp0) {
            const uint32_t bar = bar_drain + 8 * (uint32_t)(warp - 1);
            umma_commit(bar);
            for (int i = 0; i < (1 << 20) && !mbar_try_wait(bar, 0); ++i) {}
        }
        tc_fence_before();
        __syncthreads();
        tc_fence_after();
    }
    // Tensor memory and the peers' view of this CTA's shared memory are not needed by the reduction: free the one and
    // arrive on the cluster barrier now (no CTA of a cluster may leave while a peer may still read its shared memory or
    // arrive on its barriers -- all of that happens in the roles above); the wait is at the very end, when every peer
    // has long arrived.  (Both used to sit behind the reduction: about a microsecond between the last output row and
    // the exit.)
    if (warp == kMainWarps) tmem_dealloc(tmem_base, kFusedTmemCols);
    if (late_wait && !(warp >= kEpiWarp0 && warp < kEpiWarp0 + 4)) cluster_wait();   // (pairs with the set-up's arrival; the accumulator warps have waited)
    cluster_arrive();
    if (alive && warp < kMainWarps) {
        const int QB = H / 32, n_tasks = T * QB, NP = K * IB;
        const int tpc = (n_tasks + G - 1) / G;                             // tasks of the busiest CTA
        int sp = 8;
        while (sp > 1 && sp * tpc > 8) sp >>= 1;
        const int slots = 8 / sp, slot = warp / sp, part = warp - slot * sp;
        constexpr int kRG = (SPLIT || TC >= 4) ? 3 : 1;                   // groups of eight tagged words a thread polls side by side
        // Which tasks.  Steps that cannot have more units than clusters: tasks go to the CTAs from the LAST one down -- the
        // first CTAs hold the router rows and the units, and with them the next launch's critical path; they should be the
        // first to leave (the next launch's CTAs are placed in index order as SMs free up).  Steps that can: by ticket,
        // `slots` consecutive tasks each; the first was taken by the producer when it ran out of work, the next ones are
        // taken here.  A CTA that finishes late finds the tasks gone: what the grid waits for after the last store is
        // one poll by CTAs that have been polling all along, not the whole reduction of the CTA that stored last.
        const int rc = G - 1 - cta;
        const int mine = (rc < n_tasks) ? (n_tasks - rc + G - 1) / G : 0;
        float* s_sum = s_part;                                             // [8 warps][32 rows] (the partial buffers are idle now)
        bool ok = !wt.dead;
        constexpr bool dyn = SPLIT;
        unsigned ticket = dyn ? misc[5] : 0u;
#pragma unroll 1
        for (int i0 = 0; dyn ? ((unsigned long long)ticket * (unsigned)slots < (unsigned)n_tasks) : (i0 < mine); i0 += slots) {
            bool valid;
            int task;
            unsigned seen = 0u;                   // tickets handed out so far, read now, looked at after this ticket's tasks:
            if (dyn && tid == 0) asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(P.ctrl + kDoneCnt + (tag & 1u)) : "memory");   // if none are left by then, no round trip is spent on asking
            if (dyn) { task = (int)ticket * slots + slot; valid = task < n_tasks; if (!valid) task = (int)ticket * slots; }
            else { valid = (i0 + slot < mine); task = rc + (valid ? i0 + slot : i0) * G; }
            const int t = div_small(task, QB), rb = task - t * QB;
            const unsigned long long* base = P.ypl + (size_t)t * NP * H + (size_t)rb * 32 + lane;
            float acc = 0.f;
            // kRG groups of eight tagged words per thread and chunk.  The groups are polled in turn WITHOUT waiting for one
            // to complete before the next is looked at: by the time the slowest producer's words arrive, every other word
            // has been taken, and only the groups that still miss something cost another round trip.  (Waiting group by
            // group cost a round trip per group after the last arrival.)  Values are kept, summed in fixed order.
#pragma unroll 1
            for (int p0 = part; p0 < NP && ok && valid; p0 += sp * 8 * kRG) {
                float val[kRG][8];
                unsigned pend[kRG];
#pragma unroll
                for (int g = 0; g < kRG; ++g) {
                    pend[g] = 0u;
#pragma unroll
                    for (int j = 0; j < 8; ++j) { val[g][j] = 0.f; if (p0 + sp * (g * 8 + j) < NP) pend[g] |= 1u << j; }
                }
                for (uint32_t it = 1;; ++it) {
                    unsigned any = 0u;
#pragma unroll
                    for (int g = 0; g < kRG; ++g) {
                        if (pend[g]) {
                            unsigned long long v[8];
#pragma unroll
                            for (int j = 0; j < 8; ++j) if (pend[g] & (1u << j)) v[j] = ld_relaxed_u64(base + (size_t)(p0 + sp * (g * 8 + j)) * H);
#pragma unroll
                            for (int j = 0; j < 8; ++j)
                                if ((pend[g] & (1u << j)) && (unsigned)(v[j] >> 32) == tag) { pend[g] &= ~(1u << j); val[g][j] = __uint_as_float((unsigned)v[j]); }
                            any |= pend[g];
                        }
                    }
                    if (!any) break;
                    if ((it & 63u) == 0 && wt.expired(33)) { ok = false; break; }
                }
                if (!ok) break;
#pragma unroll
                for (int g = 0; g < kRG; ++g)
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        if (p0 + sp * (g * 8 + j) < NP) acc = fmaf(s_w[t * K + div_small(p0 + sp * (g * 8 + j), IB)], val[g][j], acc);
            }
            s_sum[warp * 32 + lane] = acc;
            ok = named_bar_and(2, kMain, ok);
            if (!ok) break;
            if (part == 0 && valid) {
                float r = s_sum[warp * 32 + lane];
                for (int q2 = 1; q2 < sp; ++q2) r += s_sum[(warp + q2) * 32 + lane];
                P.out[(size_t)t * H + rb * 32 + lane] = __float2bfloat16_rn(r);
            }
            if (dyn && tid == 0) misc[5] = ((unsigned long long)seen * (unsigned)slots >= (unsigned)n_tasks) ? 0xFFFFFFFFu : atomicAdd(P.ctrl + kDoneCnt + (tag & 1u), 1u);
            named_bar_sync(2, kMain);
            if (dyn) ticket = misc[5];
        }
        if (tid == 0) MOE_STAMP(13);
    }

    // ------------------------------------------------------------------ teardown
    // (every thread of the cluster arrived on the cluster barrier right after its roles: nobody waits here for long)
    cluster_wait();
    if (tid == 0) {
        if (P.stamps) { unsigned smid; asm volatile("mov.u32 %0, %%smid;" : "=r"(smid)); P.stamps[(size_t)blockIdx.x * kStampsPerCta + 14] = smid; }
        MOE_STAMP(15);
        // Open the next epoch.  CTA 0 alone does it: it got here only after every CTA of the grid had counted its share
        // of the quantised input, that is after every CTA had read this launch's tag.  (Unconditionally: a launch that
        // gave up must not leave its tag to the next one.)
        if (cta == 0) st_release(P.ctrl + kEpoch, tag);
    }
}

}  // namespace moe
