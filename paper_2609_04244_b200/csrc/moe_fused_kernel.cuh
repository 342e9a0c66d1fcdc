// Fused-unit variant of the routed-MoE decode kernel for 1..8 tokens (sm_100a).
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
//     intermediate tile needs no broadcast.  Units go to clusters round-robin; inside a cluster the stream is
//     software-pipelined by one unit (up(0) up(1) down(0) up(2) down(1) ...), so the exchange of unit i hides under
//     the gate/up tiles of unit i+1.
//   * Router (Section 3.3): CTA c computes the logits of experts c, c+G, ... for all tokens with plain FMAs (the
//     rows were prefetched into L2 before the wait on the previous launch) and publishes each as one 64-bit word
//     {launch tag, logit}; every CTA polls those words directly -- one store trip plus one load trip, no counter,
//     no fence -- and selects for all tokens itself.
//   * Input quantisation (Section 4.1) is spread over the grid into the workspace and consumed by bulk-tensor copies,
//     behind an arrival counter that is off the critical path (the first activation tile is needed a first-tile
//     latency after the first weight request).
//   * Shared memory stays below half an SM and tensor memory at 256 columns, so the CTAs of the NEXT launch
//     (programmatic dependent launch) are resident, initialised and have their router rows in L2 while this launch
//     still streams (Section 3.3 carries its lookahead across expert boundaries; this carries it across launches).
//
// Warp roles as in moe_kernel.cuh: warp 0 weight-tile producer, warp 2 activation-tile producer, warps 1 and 3
// tcgen05 MMA issuers (alternate accumulation groups), warps 4..7 accumulator/epilogue (thread = weight row).
#pragma once

#include "moe_kernel.cuh"

namespace moe {

constexpr int kFusedN = 16;                                   // MMA N of the fused variants (tokens 0..7 are columns 0..7)
constexpr int kFusedStage = kATileBytes + kFusedN * kBlock;    // weight tile + activation tile
constexpr int kFusedTmemCols = 256;                            // 8 accumulator buffers x (gate 16 + up 16) columns
constexpr int kFusedMaxRows = 4;                               // router rows per CTA: ceil(kMaxExperts / 128)

// ---------------------------------------------------------------------------------------------
// cluster / distributed-shared-memory wrappers
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t cluster_ctarank() { uint32_t r; asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r)); return r; }
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
    L.part_off = o; o += 2 * 2 * TC * kBlock * 4;              // this CTA's partial gate/up sums [slot][gate TC | up TC][128 rows]
    L.bar_off = o;  o += (3 * kMaxStages + 2 * kMaxTmemBufs + 12) * 8;
    L.misc_off = o; o += 64;
    L.ids_off = o;  o += T * K * 4;
    L.w_off = o;    o += T * K * 4;
    o = (o + 7) & ~7;
    L.mask_off = o; o += E * 16;
    L.act_off = o;  o += (E + 1) * 4;
    L.uidx_off = o; o += E * 4;
    o = (o + 15) & ~15;
    L.xs_off = o;   o += ((T + 3) & ~3) * (H / kBlock) * 4;    // input activation scales [H/128][T rounded up to 4]
    L.red_off = o;  o += 8 * kFusedMaxRows * 8 * 4;            // router partial dot products [warp][row][token]; later the amax scratch
    L.poff_off = o; o += E * 4;
    L.pair_off = o; o += ((T * K * 2 + 15) & ~15);
    L.total = o;
    return L;
}

// ---------------------------------------------------------------------------------------------
// the kernel.  TC = token columns the accumulator warps read (1, 2, 4, 8 >= T).
// ---------------------------------------------------------------------------------------------
template <int TC>
__global__ void __launch_bounds__(256, 2)
moe_fused_kernel(const __grid_constant__ CUtensorMap tmW13, const __grid_constant__ CUtensorMap tmW2,
                 const __grid_constant__ CUtensorMap tmXq, const __grid_constant__ Params P) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);

    constexpr int N = kFusedN;
    constexpr int kThreads = 256, kWarps = 8, kEpiThreads = 128;
    constexpr int kTmemBufs = 8;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int cta = blockIdx.x, G = gridDim.x;
    const int C = (int)cluster_nctarank(), rank = (int)cluster_ctarank();
    const int cl = cta / C, nCl = G / C;                         // clusters are consecutive CTAs of a 1-D grid
    const int T = P.T, H = P.H, E = P.E, I = P.I, K = P.K;
    const int KBu = H / kBlock, IB = I / kBlock, HB = H / kBlock;
    const int S = P.stages;
    const FusedSmem L = fused_smem_layout(TC, T, K, E, H, S);
    const int TS = (T + 3) & ~3;

    uint64_t* bars = (uint64_t*)(smem + L.bar_off);
    const uint32_t bar_full = smem_u32(bars), bar_empty = smem_u32(bars + kMaxStages), bar_fullb = smem_u32(bars + 2 * kMaxStages);
    const uint32_t bar_tfull = smem_u32(bars + 3 * kMaxStages), bar_tempty = smem_u32(bars + 3 * kMaxStages + kMaxTmemBufs);
    const uint32_t bar_x = smem_u32(bars + 3 * kMaxStages + 2 * kMaxTmemBufs);
    const uint32_t bar_hq = bar_x, bar_xfull = bar_x + 16, bar_xfree = bar_x + 32, bar_drain = bar_x + 48;   // 2 + 2 + 2 + 2 (+ spare)
    uint32_t* misc = (uint32_t*)(smem + L.misc_off);   // [0] tmem base, [1] U, [2] alive, [3] accumulator give-up, [4],[5] groups issued by the two MMA issuers
    int* s_ids = (int*)(smem + L.ids_off);
    float* s_w = (float*)(smem + L.w_off);
    unsigned long long* s_mask = (unsigned long long*)(smem + L.mask_off);
    int* s_act = (int*)(smem + L.act_off);
    int* s_uidx = (int*)(smem + L.uidx_off);
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
        for (int s = 0; s < S; ++s) { mbar_init(bar_full + 8 * s, 1); mbar_init(bar_fullb + 8 * s, 1); mbar_init(bar_empty + 8 * s, 1); }
        for (int b = 0; b < kTmemBufs; ++b) { mbar_init(bar_tfull + 8 * b, 1); mbar_init(bar_tempty + 8 * b, 4); }
        for (int b = 0; b < 2; ++b) {
            mbar_init(bar_hq + 8 * b, 1);
            mbar_init(bar_xfull + 8 * b, 4 * C);             // one arrival per accumulator warp of every CTA of the cluster
            mbar_init(bar_xfree + 8 * b, 4 * C);
            mbar_init(bar_drain + 8 * b, 1);
        }
        misc[3] = 0u; misc[4] = 0u; misc[5] = 0u;
        fence_barrier_init();
    }
    if (warp == 1) { tmem_alloc(smem_u32(misc), kFusedTmemCols); tmem_relinquish(); }
#pragma unroll 1
    for (int e = tid; e < 2 * E; e += kThreads) s_mask[e] = 0ull;
    // This CTA's router rows: ask L2 for them now.  (Weights are not written by the previous launch, and a prefetch
    // reads nothing into the SM.)
#pragma unroll 1
    for (int e = cta; e < E; e += G)
        for (int l = tid; l < H / 64; l += kThreads) prefetch_l2(reinterpret_cast<const char*>(P.Wr + (size_t)e * H) + l * 128);
    if (P.bias && tid * 32 < E) prefetch_l2(P.bias + tid * 32);
    // every CTA of the cluster has initialised its barriers before anyone arrives on them remotely
    cluster_arrive();
    cluster_wait();
    asm volatile("griddepcontrol.wait;" ::: "memory");

    Waiter wt;
    wt.init(P.ctrl, P.timeout_ns);
    const unsigned tag = ld_acquire(P.ctrl + kEpoch) + 1u;
    const unsigned par = tag & 1u;
    if (tid == 0) MOE_STAMP(0);
    // counters of the other launch parity start from zero next time (this launch counts in its own)
    if (cta == 0 && tid == 0) {
        P.ctrl[kRouteCnt + (par ^ 1u)] = 0u; P.ctrl[kRouteCnt2 + (par ^ 1u)] = 0u;
        P.ctrl[kQuantCnt + (par ^ 1u)] = 0u; P.ctrl[kDoneCnt + (par ^ 1u)] = 0u;
    }
#pragma unroll 1
    for (int e = cta * kThreads + tid; e < kMaxPasses * E; e += G * kThreads) P.e_cnt[(par ^ 1u) * kMaxPasses * E + e] = 0u;

    // ------------------------------------------------------------------ router logits of this CTA's experts (Section 3.3)
    {
        const int chunks = H / 8;                                 // 16-byte chunks per row
        int nrows = 0;
#pragma unroll 1
        for (int e = cta; e < E; e += G, ++nrows) {
            float acc[TC];
#pragma unroll
            for (int t = 0; t < TC; ++t) acc[t] = 0.f;
            const uint4* wrow = reinterpret_cast<const uint4*>(P.Wr + (size_t)e * H);
#pragma unroll 2
            for (int c = tid; c < chunks; c += kThreads) {
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
                if (lane == 0) s_red[(warp * kFusedMaxRows + nrows) * 8 + t] = acc[t];
            }
        }
        __syncthreads();
        if (tid < nrows * TC) {
            const int r = tid / TC, t = tid - r * TC;
            if (t < T) {
                float v = 0.f;
#pragma unroll
                for (int w = 0; w < kWarps; ++w) v += s_red[(w * kFusedMaxRows + r) * 8 + t];
                st_relaxed_u64(P.ll + (size_t)t * E + cta + r * G, ((unsigned long long)tag << 32) | (unsigned long long)__float_as_uint(v));
            }
        }
        if (tid == 0) MOE_STAMP(1);
    }
    // ------------------------------------------------------------------ input quantisation (Section 4.1), spread over the grid
    {
        const int groups = T * KBu;
#pragma unroll 1
        for (int p = (G - 1 - cta) * kWarps + warp; p < groups; p += G * kWarps) {   // from the last CTA down: the first ones have router rows
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
        fence_proxy_async();                                    // generic writes of xq -> the async proxy (bulk-tensor copies) of every CTA
        __syncthreads();
        if (tid == 0) { red_release_add(P.ctrl + kQuantCnt + par, 1u); MOE_STAMP(2); }
    }
    const uint32_t tmem_base = misc[0];

    // ------------------------------------------------------------------ gather all logits: poll the tagged words themselves
    uint32_t* s_key = reinterpret_cast<uint32_t*>(smem);
    float* s_val = reinterpret_cast<float*>(smem) + T * E;
    bool alive;
    {
        const bool softmax = (P.scoring == 0);
        bool ok = true;
#pragma unroll 1
        for (int p0 = tid; p0 < T * E && ok; p0 += 8 * kThreads) {          // eight words in flight per thread
            unsigned long long v[8];
            unsigned pending = 0u;
#pragma unroll
            for (int j = 0; j < 8; ++j) if (p0 + j * kThreads < T * E) pending |= 1u << j;
            for (uint32_t it = 1; pending; ++it) {
#pragma unroll
                for (int j = 0; j < 8; ++j) if (pending & (1u << j)) v[j] = ld_relaxed_u64(P.ll + p0 + j * kThreads);
#pragma unroll
                for (int j = 0; j < 8; ++j) if ((pending & (1u << j)) && (unsigned)(v[j] >> 32) == tag) pending &= ~(1u << j);
                if (pending && (it & 63u) == 0 && wt.expired(20)) { ok = false; break; }
            }
            if (!ok) break;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int p = p0 + j * kThreads;
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
        alive = __syncthreads_and(ok && !wt.dead) != 0;
        if (tid == 0) MOE_STAMP(3);
    }

    // ------------------------------------------------------------------ top-k for every token, in every CTA (Section 4.1)
    if (alive) {
#pragma unroll 1
        for (int t = warp; t < T; t += kWarps) {
            if (E <= 128) route_select<4>(P, t, lane, s_key + t * E, s_val + t * E, s_ids, s_w, s_mask, cta == 0, true);
            else if (E <= 256) route_select<8>(P, t, lane, s_key + t * E, s_val + t * E, s_ids, s_w, s_mask, cta == 0, true);
            else route_select<16>(P, t, lane, s_key + t * E, s_val + t * E, s_ids, s_w, s_mask, cta == 0, true);
        }
    }
    __syncthreads();
    if (tid == 0) MOE_STAMP(4);
    // ------------------------------------------------------------------ routing metadata: active experts (warp 0), routed pairs (warps 4..7)
    if (alive && warp == 0) {
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
    if (alive && warp >= kEpiWarp0) {
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
    }
    __syncthreads();
    if (tid == 0) MOE_STAMP(5);
    const int U = alive ? (int)misc[1] : 0;
    const int nU = U * IB;                                       // units of this step
    const int n = (cl < nU) ? (nU - cl + nCl - 1) / nCl : 0;     // units of this cluster: cl, cl + nCl, ...
    // this CTA's share of every unit: K blocks [kb_lo, kb_hi) of the gate/up rows, row blocks [hb_lo, hb_hi) of W2
    const int kb_lo = rank * KBu / C, kb_hi = (rank + 1) * KBu / C, nk = kb_hi - kb_lo;
    const int hb_lo = (C - 1 - rank) * HB / C, hb_hi = (C - rank) * HB / C, nh = hb_hi - hb_lo;
    auto unit_of = [&](int s, int& e, int& ib) { const int u = cl + s * nCl; const int a = div_small(u, IB); ib = u - a * IB; e = s_act[a]; };

    // Stream order of this CTA (same in every role): for s = 0..n: the gate/up k-steps of unit s (if s < n), then the
    // down tiles of unit s-1 (if s >= 1).  A gate/up k-step is two stages and one accumulation group, a down tile is
    // one stage and one group.
    // ------------------------------------------------------------------ role: weight-tile producer
    if (warp == 0) {
        if (lane == 0 && alive && n > 0) {
            const uint64_t stream_once = l2_policy_evict_first();
            int cur = 0, st = 0;
            uint32_t ph = 1u;
            uint32_t dst = smem_u32(smem), full = bar_full, empty = bar_empty;
            auto put = [&](const CUtensorMap* m, int x, int y) -> bool {
                if (!wt.mbar(empty, ph, 21)) return false;
                mbar_expect_tx(full, (uint32_t)kATileBytes);
                tma_load_2d_hint(dst, m, x, y, full, stream_once);
                ++cur;
                dst += kFusedStage; full += 8; empty += 8;
                if (++st == S) { st = 0; ph ^= 1u; dst = smem_u32(smem); full = bar_full; empty = bar_empty; }
                return true;
            };
            MOE_STAMP(6);
            for (int s = 0; s <= n && !wt.dead; ++s) {
                if (s < n) {
                    int e, ib;
                    unit_of(s, e, ib);
                    for (int k = kb_lo; k < kb_hi; ++k) {
                        if (!put(&tmW13, k * kBlock, e * 2 * I + ib * kBlock)) break;
                        if (!put(&tmW13, k * kBlock, e * 2 * I + I + ib * kBlock)) break;
                    }
                }
                if (s >= 1 && !wt.dead) {
                    int e, ib;
                    unit_of(s - 1, e, ib);
                    for (int h = hb_lo; h < hb_hi; ++h)
                        if (!put(&tmW2, ib * kBlock, e * H + h * kBlock)) break;
                }
            }
            if (wt.dead) {   // give-up path: wait (bounded) for this thread's copies in flight
                for (int it = (cur > S ? cur - S : 0); it < cur; ++it)
                    for (int i = 0; i < (1 << 20) && !mbar_try_wait(bar_full + 8 * (it % S), (uint32_t)((it / S) & 1)); ++i) {}
            }
        }
        __syncwarp();
    }
    // ------------------------------------------------------------------ role: activation-tile producer
    else if (warp == 2) {
        if (lane == 0 && alive && n > 0) {
            int cur = 0, st = 0;
            uint32_t ph = 1u;
            uint32_t dst = smem_u32(smem) + kATileBytes, full = bar_fullb, empty = bar_empty;
            auto step = [&]() { ++cur; dst += kFusedStage; full += 8; empty += 8; if (++st == S) { st = 0; ph ^= 1u; dst = smem_u32(smem) + kATileBytes; full = bar_fullb; empty = bar_empty; } };
            // the quantised input of every token is in the workspace once all CTAs have counted themselves
            if (wt.flag(P.ctrl + kQuantCnt + par, (unsigned)G, 22)) {
                fence_proxy_async();
                for (int s = 0; s <= n && !wt.dead; ++s) {
                    if (s < n) {
                        for (int k = kb_lo; k < kb_hi; ++k) {
                            if (!wt.mbar(empty, ph, 23)) break;
                            mbar_expect_tx(full, (uint32_t)(N * kBlock));
                            tma_load_2d(dst, &tmXq, k * kBlock, 0, full);        // rows 0..15 of xq (tokens beyond T are never read back)
                            step();
                            if (!wt.mbar(empty, ph, 23)) break;
                            mbar_arrive(full);                                   // the up tile shares the gate stage's activation tile
                            step();
                        }
                    }
                    if (s >= 1 && !wt.dead) {
                        for (int h = hb_lo; h < hb_hi; ++h) {
                            if (!wt.mbar(empty, ph, 23)) break;
                            mbar_arrive(full);                                   // the down tile's activation operand is the on-chip intermediate tile
                            step();
                        }
                    }
                }
            }
            if (wt.dead) {
                for (int it = (cur > S ? cur - S : 0); it < cur; ++it)
                    for (int i = 0; i < (1 << 20) && !mbar_try_wait(bar_fullb + 8 * (it % S), (uint32_t)((it / S) & 1)); ++i) {}
            }
        }
        __syncwarp();
    }
    // ------------------------------------------------------------------ role: MMA issuers (alternate accumulation groups)
    // The two threads share the stage ring; as in moe_kernel.cuh each publishes how many groups it has issued and
    // neither runs S/2 or more groups ahead of the other, so a parity wait on a stage is never a lap off.
    else if (warp == 1 || warp == 3) {
        if (lane == 0 && alive && n > 0) {
            constexpr uint32_t idesc = (1u << 4) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(kBlock >> 4) << 24);
            const uint32_t ring = smem_u32(smem);
            const int who = warp >> 1;
            int st = 0, g = 0;
            uint32_t ph = 0;
            auto advance = [&](int k) { st += k; while (st >= S) { st -= S; ph ^= 1u; } };
            int other_seen = 0;
            bool first = true;
            // common head of a group: accumulator buffer free, the other issuer not too far behind
            auto head = [&]() -> bool {
                const int buf = g & (kTmemBufs - 1);
                if (!wt.mbar(bar_tempty + 8 * buf, (uint32_t)((g >> 3) & 1) ^ 1u, 24)) return false;
                const int q = g - (S >> 1);
                const int thr = ((q & 1) != who) ? q + 1 : q;
                if (other_seen < thr) {
                    volatile uint32_t* other = misc + 4 + (who ^ 1);
                    for (uint32_t i = 1; (other_seen = (int)*other) < thr; ++i)
                        if ((i & 255u) == 0 && wt.expired(25)) return false;
                }
                return true;
            };
            for (int s = 0; s <= n && !wt.dead; ++s) {
                if (s < n) {
                    for (int k = 0; k < nk && !wt.dead; ++k, ++g) {
                        if ((g & 1) != who) { advance(2); continue; }
                        if (!head()) break;
                        const int buf = g & (kTmemBufs - 1);
                        const int st0 = st;
                        const uint32_t a0 = ring + (uint32_t)st0 * (uint32_t)kFusedStage;
                        if (!wt.mbar(bar_full + 8 * st0, ph, 26) || !wt.mbar(bar_fullb + 8 * st0, ph, 26)) break;
                        const uint64_t b_desc = make_smem_desc(a0 + kATileBytes);
                        const uint32_t d = tmem_base + (uint32_t)(buf * 2 * N);
                        if (first && who == 0) { MOE_STAMP(7); first = false; }
                        tc_fence_after();
                        {
                            const uint64_t a_desc = make_smem_desc(a0);
#pragma unroll
                            for (int kk = 0; kk < 4; ++kk) umma_f8(d, a_desc + (uint64_t)(kk * 2), b_desc + (uint64_t)(kk * 2), idesc, kk > 0 ? 1u : 0u);
                        }
                        advance(1);
                        const int st1 = st;
                        if (!wt.mbar(bar_full + 8 * st1, ph, 26) || !wt.mbar(bar_fullb + 8 * st1, ph, 26)) break;
                        tc_fence_after();
                        {
                            const uint64_t a_desc = make_smem_desc(ring + (uint32_t)st1 * (uint32_t)kFusedStage);
#pragma unroll
                            for (int kk = 0; kk < 4; ++kk) umma_f8(d + N, a_desc + (uint64_t)(kk * 2), b_desc + (uint64_t)(kk * 2), idesc, kk > 0 ? 1u : 0u);
                        }
                        umma_commit(bar_empty + 8 * st0);
                        umma_commit(bar_empty + 8 * st1);
                        umma_commit(bar_tfull + 8 * buf);
                        *(volatile uint32_t*)(misc + 4 + who) = (uint32_t)(g + 1);
                        advance(1);
                    }
                }
                if (s >= 1 && !wt.dead) {
                    const int slot = (s - 1) & 1;
                    bool hq_ok = false;
                    for (int h = 0; h < nh && !wt.dead; ++h, ++g) {
                        if ((g & 1) != who) { advance(1); continue; }
                        if (!head()) break;
                        if (!hq_ok) {                      // the intermediate tile of unit s-1 is in shared memory (written by the accumulator warps)
                            if (!wt.mbar(bar_hq + 8 * slot, (uint32_t)(((s - 1) >> 1) & 1), 27)) break;
                            hq_ok = true;
                        }
                        const int buf = g & (kTmemBufs - 1);
                        const int st0 = st;
                        if (!wt.mbar(bar_full + 8 * st0, ph, 26) || !wt.mbar(bar_fullb + 8 * st0, ph, 26)) break;
                        const uint64_t a_desc = make_smem_desc(ring + (uint32_t)st0 * (uint32_t)kFusedStage);
                        const uint64_t b_desc = make_smem_desc(smem_u32(s_hq) + (uint32_t)(slot * N * kBlock));
                        const uint32_t d = tmem_base + (uint32_t)(buf * 2 * N);
                        tc_fence_after();
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk) umma_f8(d, a_desc + (uint64_t)(kk * 2), b_desc + (uint64_t)(kk * 2), idesc, kk > 0 ? 1u : 0u);
                        umma_commit(bar_empty + 8 * st0);
                        umma_commit(bar_tfull + 8 * buf);
                        *(volatile uint32_t*)(misc + 4 + who) = (uint32_t)(g + 1);
                        advance(1);
                    }
                }
            }
            if (wt.dead) {                                     // let issued MMAs retire before TMEM is released
                umma_commit(bar_drain + 8 * (uint32_t)who);
                for (int i = 0; i < (1 << 20) && !mbar_try_wait(bar_drain + 8 * (uint32_t)who, 0); ++i) {}
            }
        }
        __syncwarp();
    }
    // ------------------------------------------------------------------ role: accumulator / epilogue warps
    else if (warp >= kEpiWarp0) {
        const int q = warp & 3, row = q * 32 + lane;           // TMEM lane == weight row inside the tile
        const int etid = tid - kEpiWarp0 * 32;
        const uint32_t t_lane = tmem_base + ((uint32_t)(q * 32) << 16);
        bool first_acc = true;
        if (alive) {
            // input scales [K block][token]: behind the same counter as the quantised input
            const bool got = (etid == 0) ? wt.flag(P.ctrl + kQuantCnt + par, (unsigned)G, 28) : true;
            if (!epi_all(got, kEpiThreads)) { wt.dead = true; }
            else {
#pragma unroll 1
                for (int i = etid; i < T * KBu; i += kEpiThreads) { const int tt = div_small(i, KBu); s_xs[(i - tt * KBu) * TS + tt] = __ldcg(P.xs + i); }
                epi_bar(kEpiThreads);
            }
        }
        int g = 0;                                             // accumulation groups consumed so far
        float sc[TC];                                          // scale of the intermediate tile per token column (unit in its down phase)
#pragma unroll
        for (int c = 0; c < TC; ++c) sc[c] = 0.f;
        // Block scales of unit s for this CTA's tiles: lane l holds K block kb_lo + l (and + 32) of the gate and of the up
        // rows, and row block hb_lo + l (and + 32) of the W2 column block.  Fetched one unit ahead of their use.
        float nwg0 = 0.f, nwu0 = 0.f, nwg1 = 0.f, nwu1 = 0.f, nw2a = 0.f, nw2b = 0.f;
        auto fetch_scales = [&](int s) {
            if (s >= n) return;
            int e, ib;
            unit_of(s, e, ib);
            const float* g13 = P.W13s + ((size_t)e * 2 * IB + ib) * KBu + kb_lo;
            const float* u13 = P.W13s + ((size_t)e * 2 * IB + IB + ib) * KBu + kb_lo;
            const float* w2 = P.W2s + ((size_t)e * HB + hb_lo) * IB + ib;
            nwg0 = (lane < nk) ? __ldg(g13 + lane) : 0.f;           nwu0 = (lane < nk) ? __ldg(u13 + lane) : 0.f;
            nwg1 = (lane + 32 < nk) ? __ldg(g13 + 32 + lane) : 0.f; nwu1 = (lane + 32 < nk) ? __ldg(u13 + 32 + lane) : 0.f;
            nw2a = (lane < nh) ? __ldg(w2 + (size_t)lane * IB) : 0.f;
            nw2b = (lane + 32 < nh) ? __ldg(w2 + (size_t)(lane + 32) * IB) : 0.f;
        };
        if (alive && !wt.dead && n > 0) {
            fetch_scales(0);
            float w2a = 0.f, w2b = 0.f, pw2a = 0.f, pw2b = 0.f;   // W2 scales of the unit in its gate/up phase, and of the one in its down phase
            for (int s = 0; s <= n; ++s) {
                pw2a = w2a; pw2b = w2b;
                // ---------------- gate/up k-steps of unit s: accumulate, then park the partial sums for the cluster
                if (s < n) {
                    int e, ib;
                    unit_of(s, e, ib);
                    // block scales of this CTA's k-steps (fetched one unit ahead), handed out by shuffle
                    float wg0 = nwg0, wu0 = nwu0, wg1 = nwg1, wu1 = nwu1;
                    w2a = nw2a; w2b = nw2b;
                    fetch_scales(s + 1);
                    float accg[TC], accu[TC];
#pragma unroll
                    for (int c = 0; c < TC; ++c) { accg[c] = 0.f; accu[c] = 0.f; }
                    for (int k = 0; k < nk; ++k, ++g) {
                        const int buf = g & (kTmemBufs - 1);
                        if (!wt.mbar(bar_tfull + 8 * buf, (uint32_t)((g >> 3) & 1), 29)) misc[3] = 1u;
                        tc_fence_after();
                        if (first_acc) { if (etid == 0) MOE_STAMP(8); first_acc = false; }
                        float dg[TC], du[TC];
                        const uint32_t tcol = t_lane + (uint32_t)(buf * 2 * N);
                        tmem_ld<TC>(tcol, dg);
                        tmem_ld<TC>(tcol + N, du);
                        tmem_ld_wait();
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(bar_tempty + 8 * buf);
                        const int kl = k & 31;
                        if (k == 32) { wg0 = wg1; wu0 = wu1; }
                        const float wsg = __shfl_sync(0xffffffffu, wg0, kl), wsu = __shfl_sync(0xffffffffu, wu0, kl);
                        const float* as = s_xs + (kb_lo + k) * TS;
#pragma unroll
                        for (int c = 0; c < TC; ++c) {
                            const float a = as[c];
                            accg[c] = fmaf(dg[c], wsg * a, accg[c]);
                            accu[c] = fmaf(du[c], wsu * a, accu[c]);
                        }
                    }
                    // park: slot s & 1 of this CTA's partial buffer, free once every peer has read the unit that used it before
                    const int slot = s & 1;
                    if (s >= 2 && lane == 0) {
                        bool okw = !wt.dead;
                        for (uint32_t i = 1; okw && !mbar_try_wait_cluster(bar_xfree + 8 * slot, (uint32_t)((s >> 1) & 1) ^ 1u); ++i)
                            if ((i & 255u) == 0 && wt.expired(30)) okw = false;
                        if (!okw) misc[3] = 1u;
                    }
                    __syncwarp();
                    float* pp = s_part + slot * 2 * TC * kBlock;
#pragma unroll
                    for (int c = 0; c < TC; ++c) { pp[c * kBlock + row] = accg[c]; pp[(TC + c) * kBlock + row] = accu[c]; }
                    __syncwarp();
                    if (lane < C) mbar_arrive_cluster(map_to_rank(bar_xfull + 8 * slot, (uint32_t)lane));
                    if (s == 0 && etid == 0) MOE_STAMP(9);
                }
                // ---------------- unit s-1: gather the cluster's partial sums, SiLU*up, requantise, then its down tiles
                if (s >= 1) {
                    const int i = s - 1, slot = i & 1;
                    int e, ib;
                    unit_of(i, e, ib);
                    const float w2a = pw2a, w2b = pw2b;                     // W2 block scales of this CTA's row blocks (fetched with the unit's gate/up scales)
                    // token columns of this expert and where their down results go
                    const unsigned long long mask = s_mask[2 * e];
                    int yoff_lane = 0;
                    if (lane < TC && ((mask >> lane) & 1ull)) {
                        const unsigned pr = s_pair[s_poff[e] + __popcll(mask & ((1ull << lane) - 1ull))];
                        yoff_lane = (((int)(pr & 0xFFu) * K + (int)(pr >> 8)) * IB + ib) * H;
                    }
                    {
                        bool okw = !wt.dead;
                        for (uint32_t it = 1; okw && !mbar_try_wait_cluster(bar_xfull + 8 * slot, (uint32_t)((i >> 1) & 1)); ++it)
                            if ((it & 255u) == 0 && wt.expired(31)) okw = false;
                        if (!okw) misc[3] = 1u;
                    }
                    float a[TC];
#pragma unroll
                    for (int c = 0; c < TC; ++c) a[c] = 0.f;
                    {
                        float sg[TC], su[TC];
#pragma unroll
                        for (int c = 0; c < TC; ++c) { sg[c] = 0.f; su[c] = 0.f; }
                        const uint32_t mine = smem_u32(s_part + slot * 2 * TC * kBlock) + (uint32_t)row * 4u;
                        for (int r = 0; r < C; ++r) {                      // rank order: every CTA of the cluster gets the same sums
                            const uint32_t src = map_to_rank(mine, (uint32_t)r);
#pragma unroll
                            for (int c = 0; c < TC; ++c) {
                                if ((mask >> c) & 1ull) {                  // only tokens routed to this expert matter (uniform)
                                    sg[c] += ld_cluster_f32(src + (uint32_t)(c * kBlock * 4));
                                    su[c] += ld_cluster_f32(src + (uint32_t)((TC + c) * kBlock * 4));
                                }
                            }
                        }
                        // SiLU(gate)*up, 128-wide amax (Section 3.3)
#pragma unroll
                        for (int c = 0; c < TC; ++c) {
                            if ((mask >> c) & 1ull) {
                                a[c] = __fdiv_rn(sg[c], 1.0f + expf(-sg[c])) * su[c];
                                const uint32_t m = __reduce_max_sync(0xffffffffu, __float_as_uint(fabsf(a[c])));
                                if (lane == 0) s_red[q * 8 + c] = __uint_as_float(m);
                            }
                        }
                    }
                    __syncwarp();
                    if (lane < C) mbar_arrive_cluster(map_to_rank(bar_xfree + 8 * slot, (uint32_t)lane));   // my reads of every peer's slot are done
                    if (!epi_all(misc[3] == 0u && !wt.dead, kEpiThreads)) { wt.dead = true; break; }
                    uint8_t* hq = s_hq + slot * N * kBlock;
#pragma unroll
                    for (int c = 0; c < TC; ++c) {
                        if ((mask >> c) & 1ull) {
                            const float amax = fmaxf(fmaxf(s_red[c], s_red[8 + c]), fmaxf(s_red[16 + c], s_red[24 + c]));
                            sc[c] = __fdiv_rn(fmaxf(amax, 1e-10f), 448.0f);
                            const float2 v = make_float2(__fdiv_rn(a[c], sc[c]), 0.f);
                            // K-major, 128-byte swizzled B tile: row = token column, 16-byte chunk (row >> 4) sits at chunk ^ (column & 7)
                            hq[c * kBlock + ((((row >> 4) ^ (c & 7)) << 4) | (row & 15))] = (uint8_t)(__nv_cvt_float2_to_fp8x2(v, __NV_SATFINITE, __NV_E4M3) & 0xFF);
                        }
                    }
                    fence_proxy_async();                                   // generic writes -> the tensor core's reads
                    epi_bar(kEpiThreads);
                    if (etid == 0) { mbar_arrive(bar_hq + 8 * slot); if (i == 0) MOE_STAMP(10); }
                    // ---- down tiles of the unit: one accumulation group each, scaled and stored as the partial of (token, slot, ib)
                    for (int h = 0; h < nh; ++h, ++g) {
                        const int buf = g & (kTmemBufs - 1);
                        if (!wt.mbar(bar_tfull + 8 * buf, (uint32_t)((g >> 3) & 1), 32)) misc[3] = 1u;
                        tc_fence_after();
                        float d[TC];
                        tmem_ld<TC>(t_lane + (uint32_t)(buf * 2 * N), d);
                        tmem_ld_wait();
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(bar_tempty + 8 * buf);
                        const float ws = __shfl_sync(0xffffffffu, (h < 32) ? w2a : w2b, h & 31);
                        float* yrow = P.yp + (size_t)(hb_lo + h) * kBlock + row;
#pragma unroll
                        for (int c = 0; c < TC; ++c) {
                            const int yo = __shfl_sync(0xffffffffu, yoff_lane, c);
                            if ((mask >> c) & 1ull) __stcg(yrow + (size_t)yo, d[c] * (ws * sc[c]));
                        }
                    }
                }
            }
        }
        // every partial of this CTA is stored: count it done (all CTAs count, with or without units)
        epi_bar(kEpiThreads);
        if (etid == 0) { if (alive && !wt.dead && misc[3] == 0u) red_release_add(P.ctrl + kDoneCnt + par, 1u); MOE_STAMP(11); }
        // ---------------- final weighted reduction (Section 3.2: only this remains in the drain); deterministic.
        // Task = (token, 128-row block), task = cta + i * G.  Warp q takes the partials p = q, q + 4, ... of the
        // K * I/128 (slot, ib) partials, four rows per lane; the four warps' sums are combined in fixed order.
        if (alive) {
            const bool got = (etid == 0) ? wt.flag(P.ctrl + kDoneCnt + par, (unsigned)G, 33) : true;
            if (!epi_all(got && !wt.dead && misc[3] == 0u, kEpiThreads)) wt.dead = true;
            if (etid == 0) MOE_STAMP(12);
            const int n_tasks = T * HB, NP = K * IB;
            float4* s_sum = reinterpret_cast<float4*>(s_part);             // [4 warps][32 lanes] (the partial buffers are idle now)
#pragma unroll 1
            for (int task = cta; task < n_tasks && !wt.dead; task += G) {
                const int t = div_small(task, HB), hb = task - t * HB;
                const float* base = P.yp + (size_t)t * K * IB * H + (size_t)hb * kBlock + lane * 4;
                float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 1
                for (int p0 = q; p0 < NP; p0 += 4 * 8) {                   // eight 16-byte loads in flight per thread
                    float4 v[8];
                    float wv[8];
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const int p = p0 + 4 * j;
                        const bool on = p < NP;
                        v[j] = on ? __ldcg(reinterpret_cast<const float4*>(base + (size_t)p * H)) : make_float4(0.f, 0.f, 0.f, 0.f);
                        wv[j] = on ? s_w[t * K + div_small(p, IB)] : 0.f;
                    }
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        acc.x = fmaf(wv[j], v[j].x, acc.x); acc.y = fmaf(wv[j], v[j].y, acc.y);
                        acc.z = fmaf(wv[j], v[j].z, acc.z); acc.w = fmaf(wv[j], v[j].w, acc.w);
                    }
                }
                s_sum[q * 32 + lane] = acc;
                epi_bar(kEpiThreads);
                if (q == 0) {
                    const float4 a0 = s_sum[lane], a1 = s_sum[32 + lane], a2 = s_sum[64 + lane], a3 = s_sum[96 + lane];
                    const float r0 = (a0.x + a1.x) + (a2.x + a3.x), r1 = (a0.y + a1.y) + (a2.y + a3.y);
                    const float r2 = (a0.z + a1.z) + (a2.z + a3.z), r3 = (a0.w + a1.w) + (a2.w + a3.w);
                    __nv_bfloat162 lo = __floats2bfloat162_rn(r0, r1), hi = __floats2bfloat162_rn(r2, r3);
                    uint2 o;
                    o.x = *reinterpret_cast<uint32_t*>(&lo);
                    o.y = *reinterpret_cast<uint32_t*>(&hi);
                    *reinterpret_cast<uint2*>(P.out + (size_t)t * H + hb * kBlock + lane * 4) = o;
                }
                epi_bar(kEpiThreads);
            }
            if (etid == 0) MOE_STAMP(13);
        }
    }

    // ------------------------------------------------------------------ teardown
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == 1) tmem_dealloc(tmem_base, kFusedTmemCols);
    // no CTA of the cluster leaves while a peer may still read its shared memory or arrive on its barriers
    cluster_arrive();
    cluster_wait();
    if (tid == 0) {
        if (P.stamps) { unsigned smid; asm volatile("mov.u32 %0, %%smid;" : "=r"(smid)); P.stamps[(size_t)blockIdx.x * kStampsPerCta + 14] = smid; }
        MOE_STAMP(15);
        __threadfence();
        const unsigned old = atomicAdd(P.ctrl + kExitCnt, 1u);
        if (old == (unsigned)G - 1u) {          // last CTA out: open the next epoch
            P.ctrl[kExitCnt] = 0u;
            __threadfence();
            st_release(P.ctrl + kEpoch, tag);
        }
    }
}

}  // namespace moe
