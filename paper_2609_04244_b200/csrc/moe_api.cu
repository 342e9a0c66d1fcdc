// Host side of the C ABI declared in include/moe_b200.h: plan, workspace layout, TMA descriptors, launch.
#include "moe_kernel.cuh"
#include "moe_fused_kernel.cuh"

#include <cstdarg>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <vector>

#include "../../include/moe_b200.h"

namespace {

thread_local char g_err[512] = "";

int fail(int code, const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
    return code;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    });
    return fn;
}

// 2-D byte tensor [rows, cols] (cols contiguous), box = box_rows x 128 bytes, 128-byte swizzle.
bool encode_2d(CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {cols};
    cuuint32_t box[2] = {128, box_rows};
    cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

constexpr int kFusedMaxT = 16;      // the fused-unit variants take up to 16 tokens (one MMA N)

struct WsLayout {
    size_t ctrl, e_cnt, dn_flag, pu_flag, pd_flag, flags_end;   // zero-initialised region = [0, flags_end)
    size_t stamps, logits, lpart, ids, wts, xs, xq, hq, hs, part_up, part_dn, y, stage_in, stage_out, ll, yp, xsl, total;
};

struct MapKey {
    const void* ptr;
    uint64_t rows, cols;
    uint32_t box_rows;
    bool operator==(const MapKey& o) const { return ptr == o.ptr && rows == o.rows && cols == o.cols && box_rows == o.box_rows; }
};

}  // namespace

struct moe_plan {
    int H, E, I, K, scoring, renorm;
    float routed_scale;
    int device, sms, smem_optin;
    unsigned long long timeout_ns;
    // schedule knobs (Section 3.4: fixed ahead of time; moe_plan_set_knob / the offline tuner change them)
    int split_weight[moe::kMaxTokens + 1];      // compacted variants: per-column cost in the range split, quarters of the fitted weight (0 off .. 8; -1 = library's choice)
    int split_slack_kib[moe::kMaxTokens + 1];   // per token count: whole units vs split-K (see range_quantum)
    int route_all_tokens[moe::kMaxTokens + 1];  // per token count: largest T for which every CTA routes all tokens
    int stages_cap[moe::kMaxTokens + 1];        // per token count: 0 = as many pipeline stages as shared memory holds
    int compact_min = 9;            // fewest tokens for which the tokens are compacted per expert
    int use_pdl = 1;                // programmatic dependent launch
    int auto_stages = 1;            // stage-ring depth by default_stages() where the knob is 0 (MOE_B200_AUTO_STAGES=0: always all that fit)
    // fused-unit variants (1..16 tokens, moe_fused_kernel.cuh)
    int fused_knob[kFusedMaxT + 1];  // per token count 1..16: 1 = the fused variant, 0 = the general one, -1 = the library's choice
    int cluster_knob[kFusedMaxT + 1];   // CTAs per unit for T = 1..16; 0 = the library's choice
    int max_clusters[9] = {0, 0, 0, 0, 0, 0, 0, 0, 0};   // clusters of that size that are co-resident at one CTA per SM (0: cannot be launched)
    int smem_per_sm = 0;
    int pairs_at_runtime = 1;       // fused variants: launches in pairs decide after routing whether the pairs share units (see fused_dyn)
    int split_units = 1;            // fused variants: equal ranges of the group list per cluster (units may be split between two clusters)
    int host_direct = 1;            // moe_forward_host: bit 0 = write a small result straight into pinned host memory, bit 1 = read a small input in place
    int take_stamps = 0;            // kernels record their phase time stamps (diagnostics)
    int debug_skip = 0;             // test hook: readiness signals the kernel leaves out (see MOE_KNOB_DEBUG_SKIP)
    moe_plan() {
        for (int t = 0; t <= moe::kMaxTokens; ++t) { split_slack_kib[t] = t <= 8 ? 200 : 100; route_all_tokens[t] = 8; stages_cap[t] = 0; split_weight[t] = -1; }
        for (int t = 0; t <= kFusedMaxT; ++t) { fused_knob[t] = -1; cluster_knob[t] = 0; }
    }
    std::mutex mu;
    std::vector<std::pair<MapKey, CUtensorMap>> maps;   // small cache of encoded descriptors

    // More than 8 tokens: the kernel compacts the tokens of each expert into the MMA columns -- 16 columns while an
    // expert sees at most 8 tokens on average, 32 columns up to 20 on average (or whenever T <= 32); denser routing
    // of more than 32 tokens takes all tokens as columns (N = 64).
    int n_hw(int T) const {
        if (T < compact_min || (long long)T * K <= 8ll * E) return 16;
        return (T <= 32 || (long long)T * K <= 20ll * E) ? 32 : 64;
    }
    bool compact(int T) const { return T >= compact_min && n_hw(T) <= 32; }
    // ranges of equal weight (instead of equal k-step counts) where tokens are compacted and experts can be crowded
    // (its set-up costs about a microsecond; it pays from two dozen tokens on, earlier where the experts' slices are
    // so short -- I <= 256 -- that the per-column epilogue work is a large share of a unit)
    int split_weight_for(int T) const {
        if (!compact(T)) return 0;
        if (split_weight[T] >= 0) return split_weight[T];
        return (T >= 24 || (T >= 16 && I <= 256)) ? 4 : 0;
    }
    bool weighted(int T) const { return split_weight_for(T) > 0; }
    int nr(int T) const { const int N = n_hw(T); return compact(T) ? (T + N - 1) / N * N : N; }   // token rows per expert in hq / hs
    // tokens per launch: 128 while 128 tokens can still be compacted (sparse routing), otherwise 64
    int chunk() const { return compact(moe::kMaxTokens) ? moe::kMaxTokens : 64; }
    int cap(int T) const { return T < chunk() ? T : chunk(); }

    WsLayout layout(int T_max) const { return layout(T_max, fused(cap(T_max))); }
    WsLayout layout(int T_max, bool with_fused) const {
        const int Tc = cap(T_max), N = n_hw(Tc), NR = nr(Tc), G = sms;
        WsLayout L;
        size_t o = 0;
        L.ctrl = o;     o += moe::kCtrlWords * 4;
        L.e_cnt = o;    o += align_up((size_t)2 * moe::kMaxPasses * E * 4, 256);
        L.dn_flag = o;  o += align_up((size_t)G * 4, 256);
        L.pu_flag = o;  o += align_up((size_t)G * 4, 256);
        L.pd_flag = o;  o += align_up((size_t)G * 4, 256);
        L.flags_end = o;
        L.stamps = o;   o += align_up((size_t)G * moe::kStampsPerCta * 8, 256);
        L.logits = o;   o += align_up((size_t)Tc * E * 4, 256);
        L.lpart = o;    o += align_up((size_t)8 * Tc * E * 4, 256);
        L.ids = o;      o += align_up((size_t)Tc * K * 4, 256);
        L.wts = o;      o += align_up((size_t)Tc * K * 4, 256);
        L.xs = o;       o += align_up((size_t)Tc * (H / 128) * 4, 256);
        L.xq = o;       o += align_up((size_t)moe::kMaxTokens * H, 1024);
        L.hq = o;       o += align_up((size_t)E * NR * I, 1024);
        L.hs = o;       o += align_up((size_t)E * NR * (I / 128) * 4, 256);
        L.part_up = o;  o += align_up((size_t)G * 2 * N * 128 * 4, 256);
        L.part_dn = o;  o += align_up((size_t)G * N * 128 * 4, 256);
        L.y = o;        o += align_up((size_t)Tc * K * H * 4, 256);
        L.stage_in = o;  o += align_up((size_t)Tc * H * 2, 256);    // device copies of host-resident input/output
        L.stage_out = o; o += align_up((size_t)Tc * H * 2, 256);    // (moe_forward_host)
        // fused variants: tagged router logits, and one down-projection partial per (token, slot, intermediate block)
        L.ll = o;       o += with_fused ? align_up((size_t)Tc * E * 8, 256) : 0;
        L.yp = o;       o += with_fused ? align_up((size_t)Tc * K * (I / 128) * H * 8, 256) : 0;
        L.xsl = o;      o += with_fused ? align_up((size_t)G * 2 * 2 * 16 * 128 * 8, 256) : 0; // partial sums exported between clusters: [CTA][2 pieces][2 x 16 columns][128 rows]
        L.total = o;
        return L;
    }

    // ---- fused-unit variants -------------------------------------------------------------------------------------
    static int fused_tc(int T) { return T <= 1 ? 1 : T <= 2 ? 2 : T <= 4 ? 4 : T <= 8 ? 8 : 16; }
    // shared memory that still lets two CTAs share an SM (the next launch's CTAs become resident under this one)
    int fused_smem_budget() const { const int half = smem_per_sm / 2 - 1024; return half < smem_optin ? half : smem_optin; }
    // Depth of the fused variants' stage ring when the knob is 0: all that fits -- except where a step is expected to have
    // more units than CTAs (every CTA then works through a range of several pieces): 8.  Measured: config 2 at T = 6
    // and 8 -1.1 and -1.5 us, Qwen3.5-35B at T=8 -1.6, config 4 at T=1 -1.2, config 2 at T=4 -0.4; with fewer units than
    // CTAs a shallower ring loses (config 2 T=2 +0.6, DeepSeek-V3.1 TP8 T=8 +3.3, config 5 T=1 +0.4).
    int fused_stages(int T) const {
        int cap_s = stages_cap[T];
        const long long eu = (long long)expected_experts(T) * (I / 128);
        if (cap_s <= 0 && (eu > sms || (fused_dyn(T) && long_units() && eu > sms / 2 && eu * 5 <= (long long)sms * 4))) cap_s = 8;
        const int budget = smem_optin;
        for (int s = (cap_s > 0 && cap_s < moe::kMaxStages) ? cap_s : moe::kMaxStages; s >= 2; --s)
            if (moe::fused_smem_layout(fused_tc(T), T, K, E, H, s).total + 1024 <= budget) {
                // (the library's own choice is an even depth: groups are pairs of tiles, and with an odd ring every other lap
                // has a pair that wraps around its end -- config 2 at one token: 17.3 us with 10 stages, 17.7 with 11, 17.8 with 9)
                return (stages_cap[T] <= 0 && (s & 1) && s > 2) ? s - 1 : s;
            }
        return 0;
    }
    // Expected distinct experts of a step of T tokens under uniform routing (text after Eq. 5), rounded up.
    int expected_experts(int T) const { return (int)std::ceil(E * (1.0 - std::pow(1.0 - (double)K / E, (double)T)) - 1e-9); }
    // CTAs per unit: the largest cluster size for which the expected units -- (expert, 128-wide intermediate block)
    // pairs -- still get a cluster each, so that the step is one round in which every unit's 3 * H/128 tiles are
    // shared by as many CTAs as possible; one CTA per unit once there are more units than SMs.  (Measured on the nine
    // benchmark shapes at 1-8 tokens: this is the fastest size in 47 of 54 cases and within 4 % in the others.)
    // Cluster size by the expected number of units: the largest of 4, 2 for which every unit gets a cluster of its own.
    int fused_cluster_static(int T) const {
        const int KB = H / 128;
        const long long units = (long long)expected_experts(T) * (I / 128);
        for (int C = 4; C > 1; C /= 2)
            if (max_clusters[C] > 0 && C <= KB && units <= max_clusters[C]) return C;
        return max_clusters[1] > 0 ? 1 : 0;
    }
    // Where that says 1 or 2 the launch is made in pairs that cover the whole grid, and the kernel decides after routing,
    // from the number of units the step really has, whether the CTAs of a pair share units or work alone.
    bool fused_dyn(int T) const {
        if (cluster_knob[T] != 0 || !pairs_at_runtime) return false;
        const int C = fused_cluster_static(T), KB = H / 128;
        return (C == 1 || C == 2) && KB % 2 == 0 && max_clusters[2] * 2 == sms && max_clusters[1] == sms;
    }
    // a unit of 60 accumulation groups and more (H/128 gate/up groups and half as many down groups)
    bool long_units() const { return (H / 128) * 3 / 2 >= 60; }
    int fused_cluster(int T) const {
        const int KB = H / 128;
        const int knob = cluster_knob[T];
        if (knob > 0) return (knob <= 8 && max_clusters[knob] > 0 && knob <= KB) ? knob : 0;
        return fused_dyn(T) ? 2 : fused_cluster_static(T);
    }
    int fused_grid(int T) const { const int C = fused_cluster(T); return C ? C * max_clusters[C] : 0; }
    bool fused_possible(int T) const {
        // (up to 8 tokens the compaction threshold of the general variant also says where the fused one may run: a
        // caller who lowers it asks for compaction there)
        return T >= 1 && T <= kFusedMaxT && (T > 8 || T < compact_min) && H <= 8192 && fused_cluster(T) > 0 && fused_stages(T) >= 2;
    }
    // The library's choice, by the length of the weight stream: tiles per CTA at the expected number of distinct experts.
    // The fused variant has the shorter latency chain (routing, hand-over, reduction) but its accumulator warps work
    // per group; the general variant streams longer runs at a higher rate.
    // Measured crossover on the nine benchmark shapes (1-8 tokens): about 125 tiles per CTA; about 160 where a unit's
    // down projection is at most two K blocks (there the general variant's per-unit work weighs most) and for a single
    // token.
    bool fused(int T) const {
        if (!fused_possible(T) || fused_knob[T] == 0) return false;
        if (fused_knob[T] == 1) return true;
        const double tiles = 3.0 * expected_experts(T) * (I / 128) * (H / 128) / sms;
        // 9..16 tokens: the 16-column instantiation computes every column for every unit while the general variant
        // compacts (an expert sees one or two of the tokens): it pays only where the whole step is a few tiles per CTA
        // (measured: config 1 +15..18 %; the Qwen-sized layers -15..-25 %, the TP8 shards -4..+2 %)
        if (T > 8) return tiles <= 30.0;
        return tiles <= 125.0 || ((I / 128 <= 2 || T == 1) && tiles <= 160.0);
    }

    // Default depth of the stage ring when the knob is 0.  Measured (config 2 and the paper's shapes,
    // T = 1..64, ring depths 12/10/8/6): a CTA whose whole step is a handful of tiles wants every tile requested at
    // once; short streams run 2-7 % faster on a ring of 6, medium ones 1-2 % faster on 8; long streams want all the
    // depth that fits.  "Length" = weight tiles per CTA for the expected number of distinct experts (text after Eq. 5).
    int default_stages(int T) const {
        const double U = E * (1.0 - std::pow(1.0 - (double)K / E, (double)T));
        const double tiles = 3.0 * U * (I / 128) * (H / 128) / sms;
        if (tiles <= 18.0) return 0;
        if (tiles <= 105.0) return 6;
        if (tiles <= 450.0) return 8;
        return 0;
    }

    int stages_for(int N, int T) const {
        int cap_s = stages_cap[T <= moe::kMaxTokens ? T : moe::kMaxTokens];
        if (cap_s == 0 && auto_stages) cap_s = default_stages(T);
        for (int s = (cap_s > 0 && cap_s < moe::kMaxStages) ? cap_s : moe::kMaxStages; s >= 2; --s) {
            const moe::SmemLayout L = moe::smem_layout(N, T, K, E, H, I, s, compact(T), weighted(T));
            if (L.total + 1024 <= smem_optin) return s;
        }
        return 0;
    }

    bool get_map(CUtensorMap* out, const void* ptr, uint64_t rows, uint64_t cols, uint32_t box_rows) {
        MapKey k{ptr, rows, cols, box_rows};
        std::lock_guard<std::mutex> lock(mu);
        for (auto& kv : maps)
            if (kv.first == k) { *out = kv.second; return true; }
        CUtensorMap m;
        if (!encode_2d(&m, ptr, rows, cols, box_rows)) return false;
        if (maps.size() >= 256) maps.erase(maps.begin());
        maps.emplace_back(k, m);
        *out = m;
        return true;
    }
};

using Plan = struct moe_plan;

namespace {

template <int N, int TC, bool WS = false>
int launch(Plan* p, const CUtensorMap& m13, const CUtensorMap& m2, const CUtensorMap& mx, const CUtensorMap& mh,
           const moe::Params& P, int smem_bytes, cudaStream_t stream) {
    // (the opt-in shared-memory size of every variant was set by resident<>() when the plan was made)
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(p->sms, 1, 1);
    cfg.blockDim = dim3(128 + 128 * (TC >= 32 ? 2 : 1), 1, 1);
    cfg.dynamicSmemBytes = smem_bytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // overlap our launch latency with the previous
    attr[0].val.programmaticStreamSerializationAllowed = 1;            // kernel's tail; the kernel itself waits for it
    cfg.attrs = attr;
    cfg.numAttrs = p->use_pdl ? 1 : 0;
    cudaError_t err = cudaLaunchKernelEx(&cfg, moe::moe_decode_kernel<N, TC, WS>, m13, m2, mx, mh, P);
    if (err == cudaSuccess) err = cudaGetLastError();
    if (err != cudaSuccess) return fail(MOE_ERR_CUDA, "kernel launch failed: %s", cudaGetErrorString(err));
    return MOE_OK;
}

// Fused-unit variants: grid = clusters x C CTAs, cluster size chosen at run time.
template <int TC, bool SPLIT>
int launch_fused(Plan* p, int grid, int C, const CUtensorMap& m13, const CUtensorMap& m2, const CUtensorMap& mx,
                 const moe::Params& P, int smem_bytes, cudaStream_t stream) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid, 1, 1);
    cfg.blockDim = dim3(moe::kFusedThreads, 1, 1);
    cfg.dynamicSmemBytes = smem_bytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = C; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = p->use_pdl ? 2 : 1;
    cudaError_t err = cudaLaunchKernelEx(&cfg, moe::moe_fused_kernel<TC, SPLIT>, m13, m2, mx, P);
    if (err == cudaSuccess) err = cudaGetLastError();
    if (err != cudaSuccess) return fail(MOE_ERR_CUDA, "kernel launch failed: %s", cudaGetErrorString(err));
    return MOE_OK;
}

// Clusters of C CTAs of the fused kernel that are co-resident when every SM holds ONE of its CTAs (the other half of
// the SM may still belong to the previous launch); 0 when such a cluster cannot be launched at all.
template <int TC>
int fused_clusters(int C, int smem_optin, int sms) {
    if (cudaFuncSetAttribute(moe::moe_fused_kernel<TC, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_optin) != cudaSuccess) { cudaGetLastError(); return 0; }
    if (cudaFuncSetAttribute(moe::moe_fused_kernel<TC, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_optin) != cudaSuccess) { cudaGetLastError(); return 0; }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((sms / C) * C, 1, 1);
    cfg.blockDim = dim3(moe::kFusedThreads, 1, 1);
    cfg.dynamicSmemBytes = smem_optin;                         // a footprint that admits one CTA per SM
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = C; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int n = 0;
    int m = 0;
    if (cudaOccupancyMaxActiveClusters(&n, moe::moe_fused_kernel<TC, false>, &cfg) != cudaSuccess) { cudaGetLastError(); return 0; }
    if (cudaOccupancyMaxActiveClusters(&m, moe::moe_fused_kernel<TC, true>, &cfg) != cudaSuccess) { cudaGetLastError(); return 0; }
    if (m < n) n = m;
    return n < sms / C ? n : sms / C;
}

template <int N, int TC, bool WS = false>
bool resident(int smem_optin, int smem_bytes) {
    int blocks = 0;
    if (cudaFuncSetAttribute(moe::moe_decode_kernel<N, TC, WS>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_optin) != cudaSuccess) return false;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&blocks, moe::moe_decode_kernel<N, TC, WS>, 128 + 128 * (TC >= 32 ? 2 : 1), smem_bytes) != cudaSuccess) return false;
    return blocks >= 1;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Kernel parameters for a step of T tokens on workspace `w` laid out as L.
moe::Params make_params(const Plan* p, int T, int stages, const WsLayout& L, uint8_t* w, const void* hidden, const void* Wr,
                        const float* bias, const float* W13s, const float* W2s, void* out) {
    moe::Params P;
    P.T = T; P.H = p->H; P.E = p->E; P.I = p->I; P.K = p->K; P.scoring = p->scoring; P.renorm = p->renorm;
    P.routed_scale = p->routed_scale;
    P.stages = stages;
    P.split_slack_kib = p->split_slack_kib[T];
    P.split_weight = p->split_weight_for(T);
    P.route_all_tokens = p->route_all_tokens[T];
    P.nr = p->nr(T);
    P.grid_magic = (1ull << 40) / (unsigned long long)p->sms + 1ull;
    P.timeout_ns = p->timeout_ns;
    P.hidden = static_cast<const __nv_bfloat16*>(hidden);
    P.Wr = static_cast<const __nv_bfloat16*>(Wr);
    P.bias = (p->scoring == MOE_SCORE_SIGMOID_BIAS) ? bias : nullptr;
    P.W13s = W13s; P.W2s = W2s;
    P.out = static_cast<__nv_bfloat16*>(out);
    P.ctrl = reinterpret_cast<unsigned*>(w + L.ctrl);
    P.logits = reinterpret_cast<float*>(w + L.logits);
    P.lpart = reinterpret_cast<float*>(w + L.lpart);
    P.ids = reinterpret_cast<int*>(w + L.ids);
    P.wts = reinterpret_cast<float*>(w + L.wts);
    P.xq = w + L.xq;
    P.xs = reinterpret_cast<float*>(w + L.xs);
    P.hq = w + L.hq;
    P.hs = reinterpret_cast<float*>(w + L.hs);
    P.e_cnt = reinterpret_cast<unsigned*>(w + L.e_cnt);
    P.dn_flag = reinterpret_cast<unsigned*>(w + L.dn_flag);
    P.part_up = reinterpret_cast<float*>(w + L.part_up);
    P.part_dn = reinterpret_cast<float*>(w + L.part_dn);
    P.pu_flag = reinterpret_cast<unsigned*>(w + L.pu_flag);
    P.pd_flag = reinterpret_cast<unsigned*>(w + L.pd_flag);
    P.y = reinterpret_cast<float*>(w + L.y);
    P.ll = reinterpret_cast<unsigned long long*>(w + L.ll);
    P.ypl = reinterpret_cast<unsigned long long*>(w + L.yp);
    P.xsl = reinterpret_cast<unsigned long long*>(w + L.xsl);
    P.fsplit = 0;
    P.fC = 1; P.fnCl = p->sms; P.fdyn = 0; P.grid_magic1 = 0;
    for (int r = 0; r < 9; ++r) { P.fkb[r] = 0; P.fhb[r] = 0; }
    P.stamps = p->take_stamps ? reinterpret_cast<unsigned long long*>(w + L.stamps) : nullptr;
    P.stamps_buf = reinterpret_cast<unsigned long long*>(w + L.stamps);
    P.stamps_fine = p->take_stamps >= 2;
    P.debug_skip = p->debug_skip;
    return P;
}

// Pick the kernel variant for T tokens: (MMA N, token columns read by the accumulator warps).
int dispatch(Plan* p, int T, const CUtensorMap& m13, const CUtensorMap& m2, const CUtensorMap& mx,
             const CUtensorMap& mh, const moe::Params& P, int smem_bytes, cudaStream_t stream) {
    if (!p->compact(T)) {
        if (T == 1) return launch<16, 1>(p, m13, m2, mx, mh, P, smem_bytes, stream);
        if (T == 2) return launch<16, 2>(p, m13, m2, mx, mh, P, smem_bytes, stream);
        if (T <= 4) return launch<16, 4>(p, m13, m2, mx, mh, P, smem_bytes, stream);
        if (T <= 8) return launch<16, 8>(p, m13, m2, mx, mh, P, smem_bytes, stream);
    }
    if (p->weighted(T)) {
        if (p->n_hw(T) == 16) return launch<16, 16, true>(p, m13, m2, mx, mh, P, smem_bytes, stream);
        return launch<32, 32, true>(p, m13, m2, mx, mh, P, smem_bytes, stream);
    }
    if (p->n_hw(T) == 16) return launch<16, 16>(p, m13, m2, mx, mh, P, smem_bytes, stream);
    if (p->n_hw(T) == 32) return launch<32, 32>(p, m13, m2, mx, mh, P, smem_bytes, stream);
    return launch<64, 64>(p, m13, m2, mx, mh, P, smem_bytes, stream);
}

// One launch: T tokens (at most the plan's tokens per launch) on workspace `ws` laid out as `L`.  `fused` selects the
// fused-unit variant (L must then hold its scratch).  `cache_maps` = keep the encoded TMA descriptors in the plan.
int run_step(Plan* p, int T, bool fused, const WsLayout& L, bool cache_maps, const void* hidden, const void* Wr, const float* bias,
             const void* W13, const float* W13s, const void* W2, const float* W2s, void* out, void* ws, cudaStream_t stream) {
    uint8_t* w = static_cast<uint8_t*>(ws);
    auto map = [&](CUtensorMap* m, const void* ptr, uint64_t rows, uint64_t cols, uint32_t box_rows) {
        return cache_maps ? p->get_map(m, ptr, rows, cols, box_rows) : encode_2d(m, ptr, rows, cols, box_rows);
    };
    CUtensorMap m13, m2, mx, mh;
    if (fused) {
        const int TC = Plan::fused_tc(T), C = p->fused_cluster(T), grid = p->fused_grid(T), stages = p->fused_stages(T);
        if (C < 1 || grid < C || stages < 2) return fail(MOE_ERR_OCCUPANCY, "the fused variant cannot be launched for T=%d", T);
        if (!map(&m13, W13, (uint64_t)p->E * 2 * p->I, p->H, 128) || !map(&m2, W2, (uint64_t)p->E * p->H, p->I, 128) ||
            !map(&mx, w + L.xq, moe::kMaxTokens, p->H, moe::kFusedN))
            return fail(MOE_ERR_CUDA, "cuTensorMapEncodeTiled failed");
        moe::Params P = make_params(p, T, stages, L, w, hidden, Wr, bias, W13s, W2s, out);
        const int KB = p->H / 128;
        P.fC = C; P.fnCl = grid / C;
        P.fdyn = p->fused_dyn(T) ? (p->fused_cluster_static(T) == 2 ? 1 : 2) + (p->long_units() ? 4 : 0) : 0;
        P.grid_magic1 = (1ull << 40) / (unsigned long long)grid + 1ull;
        // units are shared between clusters only where the step can have more units than clusters at all: T tokens select
        // at most min(E, T * top_k) experts (the instantiations without that code are smaller and faster)
        const int max_units = (T * p->K < p->E ? T * p->K : p->E) * (p->I / 128);
        // (pairs that may work alone: then the clusters are the CTAs)
        P.fsplit = (p->split_units && KB % C == 0 && (max_units > ((P.fdyn && !(P.fdyn & 4)) ? grid : P.fnCl) || p->split_units == 2)) ? p->split_units : 0;
        P.grid_magic = (1ull << 40) / (unsigned long long)P.fnCl + 1ull;     // the fused kernel divides by the cluster count
        for (int r = 0; r <= C; ++r) { P.fkb[r] = r * KB / C; P.fhb[C - r] = KB - r * KB / C; }   // W2 row blocks in reverse rank order: the two shares add up evenly
        const int smem = moe::fused_smem_layout(TC, T, p->K, p->E, p->H, stages).total + 1024;
        switch (TC) {
            case 1: return P.fsplit ? launch_fused<1, true>(p, grid, C, m13, m2, mx, P, smem, stream) : launch_fused<1, false>(p, grid, C, m13, m2, mx, P, smem, stream);
            case 2: return P.fsplit ? launch_fused<2, true>(p, grid, C, m13, m2, mx, P, smem, stream) : launch_fused<2, false>(p, grid, C, m13, m2, mx, P, smem, stream);
            case 4: return P.fsplit ? launch_fused<4, true>(p, grid, C, m13, m2, mx, P, smem, stream) : launch_fused<4, false>(p, grid, C, m13, m2, mx, P, smem, stream);
            case 8: return P.fsplit ? launch_fused<8, true>(p, grid, C, m13, m2, mx, P, smem, stream) : launch_fused<8, false>(p, grid, C, m13, m2, mx, P, smem, stream);
            default: return P.fsplit ? launch_fused<16, true>(p, grid, C, m13, m2, mx, P, smem, stream) : launch_fused<16, false>(p, grid, C, m13, m2, mx, P, smem, stream);
        }
    }
    const int N = p->n_hw(T);
    const int stages = p->stages_for(N, T);
    if (stages < 2) return fail(MOE_ERR_OCCUPANCY, "shared memory too small for a 2-stage pipeline");
    const moe::SmemLayout SL = moe::smem_layout(N, T, p->K, p->E, p->H, p->I, stages, p->compact(T), p->weighted(T));
    if (!map(&m13, W13, (uint64_t)p->E * 2 * p->I, p->H, 128) || !map(&m2, W2, (uint64_t)p->E * p->H, p->I, 128) ||
        !map(&mx, w + L.xq, moe::kMaxTokens, p->H, N) || !map(&mh, w + L.hq, (uint64_t)p->E * p->nr(T), p->I, N))
        return fail(MOE_ERR_CUDA, "cuTensorMapEncodeTiled failed");
    const moe::Params P = make_params(p, T, stages, L, w, hidden, Wr, bias, W13s, W2s, out);
    return dispatch(p, T, m13, m2, mx, mh, P, SL.total + 1024, stream);
}

int forward_chunk(Plan* p, int T, const void* hidden, const void* Wr, const float* bias, const void* W13,
                  const float* W13s, const void* W2, const float* W2s, void* out, void* ws, size_t ws_bytes,
                  cudaStream_t stream) {
    const bool fused = p->fused(T);
    const WsLayout L = p->layout(T, fused);
    if (ws_bytes < L.total) return fail(MOE_ERR_WORKSPACE, "workspace has %zu bytes, %zu needed for T=%d", ws_bytes, L.total, T);
    return run_step(p, T, fused, L, true, hidden, Wr, bias, W13, W13s, W2, W2s, out, ws, stream);
}

int check_forward_args(Plan* p, int T, const void* hidden, const void* Wr, const float* bias, const void* W13,
                       const float* W13s, const void* W2, const float* W2s, void* out, void* ws) {
    if (!p) return fail(MOE_ERR_ARG, "plan is NULL");
    if (T < 1) return fail(MOE_ERR_ARG, "T must be >= 1 (got %d)", T);
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev != p->device) return fail(MOE_ERR_ARG, "the plan's device (%d) must be the current device", p->device);
    if (!hidden || !Wr || !W13 || !W13s || !W2 || !W2s || !out) return fail(MOE_ERR_ARG, "a tensor pointer is NULL");
    if (!ws) return fail(MOE_ERR_WORKSPACE, "workspace is NULL");
    if (p->scoring == MOE_SCORE_SIGMOID_BIAS && bias && !aligned16(bias)) return fail(MOE_ERR_ALIGN, "sel_bias not 16-byte aligned");
    if (!aligned16(hidden) || !aligned16(Wr) || !aligned16(W13) || !aligned16(W13s) || !aligned16(W2) || !aligned16(W2s) ||
        !aligned16(out))
        return fail(MOE_ERR_ALIGN, "tensor pointers must be 16-byte aligned");
    if (reinterpret_cast<uintptr_t>(ws) & 255u) return fail(MOE_ERR_ALIGN, "workspace must be 256-byte aligned");
    return MOE_OK;
}

}  // namespace

extern "C" {

const char* moe_last_error(void) { return g_err; }

int moe_plan_set_knob(moe_plan_t plan, int T, int knob, int value) {
    if (!plan) return fail(MOE_ERR_ARG, "plan is NULL");
    if (T < 0 || T > moe::kMaxTokens) return fail(MOE_ERR_ARG, "T must be 0 (all token counts) or 1..%d", moe::kMaxTokens);
    const int lo = T ? T : 0, hi = T ? T : moe::kMaxTokens;
    switch (knob) {
        case MOE_KNOB_STAGES:
            if (value != 0 && (value < 2 || value > moe::kMaxStages)) return fail(MOE_ERR_ARG, "stages must be 0 (as many as fit) or 2..%d", moe::kMaxStages);
            for (int t = lo; t <= hi; ++t) plan->stages_cap[t] = value;
            return MOE_OK;
        case MOE_KNOB_SPLIT_SLACK_KIB:
            if (value < 0 || value > (1 << 20)) return fail(MOE_ERR_ARG, "split slack out of range");
            for (int t = lo; t <= hi; ++t) plan->split_slack_kib[t] = value;
            return MOE_OK;
        case MOE_KNOB_ROUTE_ALL_TOKENS:
            if (value < 0 || value > 64) return fail(MOE_ERR_ARG, "route-all token count must be 0..64");
            for (int t = lo; t <= hi; ++t) plan->route_all_tokens[t] = value;
            return MOE_OK;
        case MOE_KNOB_COMPACT_MIN:
            if (value < 2 || value > 9) return fail(MOE_ERR_ARG, "compaction threshold must be 2..9 tokens");
            plan->compact_min = value;
            return MOE_OK;
        case MOE_KNOB_PDL:
            plan->use_pdl = value != 0;
            return MOE_OK;
        case MOE_KNOB_SPLIT_WEIGHT:
            if (value < -1 || value > 8) return fail(MOE_ERR_ARG, "split weight must be -1 (library's choice), 0 (off) or 1..8");
            for (int t = lo; t <= hi; ++t) plan->split_weight[t] = value;
            return MOE_OK;
        case MOE_KNOB_FUSED:
            if (value < -1 || value > 1) return fail(MOE_ERR_ARG, "fused must be -1 (library's choice), 0 or 1");
            for (int t = (lo < 1 ? 1 : lo); t <= (hi > kFusedMaxT ? kFusedMaxT : hi); ++t) plan->fused_knob[t] = value;
            return MOE_OK;
        case MOE_KNOB_CLUSTER:
            if (value != 0 && value != 1 && value != 2 && value != 4 && value != 8) return fail(MOE_ERR_ARG, "cluster size must be 0 (library's choice), 1, 2, 4 or 8");
            if (value > 0 && plan->max_clusters[value] <= 0) return fail(MOE_ERR_OCCUPANCY, "clusters of %d CTAs cannot be launched on this device", value);
            for (int t = (lo < 1 ? 1 : lo); t <= (hi > kFusedMaxT ? kFusedMaxT : hi); ++t) plan->cluster_knob[t] = value;
            return MOE_OK;
        case MOE_KNOB_SPLIT_UNITS:
            if (value < 0 || value > 2) return fail(MOE_ERR_ARG, "split_units must be 0, 1 or 2");
            plan->split_units = value;
            return MOE_OK;
        case MOE_KNOB_HOST_DIRECT:
            if (value < 0 || value > 3) return fail(MOE_ERR_ARG, "host-direct must be 0..3");
            plan->host_direct = value;
            return MOE_OK;
        case MOE_KNOB_DEBUG_SKIP:
            if (value < 0 || value > 1) return fail(MOE_ERR_ARG, "debug skip must be 0 or 1");
            plan->debug_skip = value;
            return MOE_OK;
        case MOE_KNOB_STAMPS:
            if (value < 0 || value > 2) return fail(MOE_ERR_ARG, "stamps must be 0, 1 or 2");
            plan->take_stamps = value;
            return MOE_OK;
        default:
            return fail(MOE_ERR_ARG, "unknown knob %d", knob);
    }
}

int moe_plan_get_knob(moe_plan_t plan, int T, int knob, int* value) {
    if (!plan || !value) return fail(MOE_ERR_ARG, "plan or value is NULL");
    if (T < 0 || T > moe::kMaxTokens) return fail(MOE_ERR_ARG, "T must be 0..%d", moe::kMaxTokens);
    const int t = T ? T : 1;
    switch (knob) {
        case MOE_KNOB_STAGES: *value = plan->stages_cap[t]; return MOE_OK;
        case MOE_KNOB_SPLIT_SLACK_KIB: *value = plan->split_slack_kib[t]; return MOE_OK;
        case MOE_KNOB_ROUTE_ALL_TOKENS: *value = plan->route_all_tokens[t]; return MOE_OK;
        case MOE_KNOB_COMPACT_MIN: *value = plan->compact_min; return MOE_OK;
        case MOE_KNOB_PDL: *value = plan->use_pdl; return MOE_OK;
        case MOE_KNOB_SPLIT_WEIGHT: *value = plan->split_weight[t]; return MOE_OK;
        case MOE_KNOB_FUSED: *value = t <= kFusedMaxT ? plan->fused_knob[t] : 0; return MOE_OK;
        case MOE_KNOB_CLUSTER: *value = t <= kFusedMaxT ? plan->cluster_knob[t] : 0; return MOE_OK;
        case MOE_KNOB_STAMPS: *value = plan->take_stamps; return MOE_OK;
        case MOE_KNOB_DEBUG_SKIP: *value = plan->debug_skip; return MOE_OK;
        case MOE_KNOB_SPLIT_UNITS: *value = plan->split_units; return MOE_OK;
        case MOE_KNOB_HOST_DIRECT: *value = plan->host_direct; return MOE_OK;
        default: return fail(MOE_ERR_ARG, "unknown knob %d", knob);
    }
}

int moe_plan_ex(int H, int E, int I, int top_k, int scoring, int renorm, float routed_scale, moe_plan_t* out) {
    if (!out) return fail(MOE_ERR_ARG, "out is NULL");
    *out = nullptr;
    if (H <= 0 || I <= 0 || H % 128 || I % 128) return fail(MOE_ERR_SHAPE, "H and I must be positive multiples of 128");
    if (E < 1 || E > moe::kMaxExperts) return fail(MOE_ERR_SHAPE, "E must be in [1,%d]", moe::kMaxExperts);
    if (top_k < 1 || top_k > E || top_k > moe::kMaxTopK) return fail(MOE_ERR_SHAPE, "top_k must be in [1,min(E,%d)]", moe::kMaxTopK);
    if (scoring != MOE_SCORE_SOFTMAX && scoring != MOE_SCORE_SIGMOID_BIAS) return fail(MOE_ERR_ARG, "unknown scoring %d", scoring);
    {   // the kernel indexes k-steps with 32-bit integers
        const long long ks = (long long)E * (H / 128) * (I / 128);
        if (ks * 256 >= (1ll << 31) || (long long)E * 2 * I * H / 128 >= (1ll << 31))
            return fail(MOE_ERR_SHAPE, "layer too large for 32-bit k-step indices");
        // weighted range split of the compacted variants: a k-step weighs < 256, a unit list holds up to
        // E + kMaxTokens * top_k / 16 virtual experts, one virtual expert's weight goes through div_small()
        const long long per_expert = (long long)(H / 128) * (I / 128);
        if (per_expert * 256 >= (1ll << 22) || (ks + (long long)(moe::kMaxTokens * top_k / 16 + 1) * per_expert) * 256 >= (1ll << 32))
            return fail(MOE_ERR_SHAPE, "layer too large for the 32-bit range weights");
    }
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev == 0) {
        cudaGetLastError();
        return fail(MOE_ERR_UNSUPPORTED_ARCH, "no CUDA device: this library has no CPU fallback");
    }
    int dev = 0;
    cudaDeviceProp prop;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaGetDeviceProperties(&prop, dev) != cudaSuccess)
        return fail(MOE_ERR_CUDA, "cannot query the current device");
    if (prop.major != 10 || prop.minor != 0) return fail(MOE_ERR_UNSUPPORTED_ARCH, "device is sm_%d%d; this library is built for sm_100a only", prop.major, prop.minor);
    Plan* p = new Plan();
    p->H = H; p->E = E; p->I = I; p->K = top_k; p->scoring = scoring; p->renorm = renorm ? 1 : 0;
    p->routed_scale = routed_scale;
    p->device = dev;
    p->sms = prop.multiProcessorCount < moe::kMaxGrid ? prop.multiProcessorCount : moe::kMaxGrid;   // one CTA per SM, up to the size of the kernel's range tables
    p->smem_optin = (int)prop.sharedMemPerBlockOptin;
    p->smem_per_sm = (int)prop.sharedMemPerMultiprocessor;
    p->timeout_ns = 1000ull * 1000ull * 1000ull;
    // schedule overrides for experiments (the paper tunes its schedule offline, Section 3.4)
    // environment overrides for experiments (the same knobs moe_plan_set_knob sets)
    if (const char* v = getenv("MOE_B200_STAGES")) moe_plan_set_knob(p, 0, MOE_KNOB_STAGES, atoi(v));
    if (const char* v = getenv("MOE_B200_PDL")) moe_plan_set_knob(p, 0, MOE_KNOB_PDL, atoi(v));
    if (const char* v = getenv("MOE_B200_AUTO_STAGES")) p->auto_stages = atoi(v) != 0;
    if (const char* v = getenv("MOE_B200_SPLIT_SLACK_KIB")) moe_plan_set_knob(p, 0, MOE_KNOB_SPLIT_SLACK_KIB, atoi(v));
    if (const char* v = getenv("MOE_B200_COMPACT_MIN")) moe_plan_set_knob(p, 0, MOE_KNOB_COMPACT_MIN, atoi(v));
    if (const char* v = getenv("MOE_B200_SPLIT_WEIGHT")) moe_plan_set_knob(p, 0, MOE_KNOB_SPLIT_WEIGHT, atoi(v));
    if (const char* v = getenv("MOE_B200_ROUTE_ALL")) moe_plan_set_knob(p, 0, MOE_KNOB_ROUTE_ALL_TOKENS, atoi(v));
    // fused-unit variants: which cluster sizes can be co-resident (Section 3.2: the realised occupancy is checked, not assumed)
    for (int C = 1; C <= 8; C *= 2) {
        const int n1 = fused_clusters<1>(C, p->smem_optin, p->sms), n2 = fused_clusters<2>(C, p->smem_optin, p->sms);
        const int n4 = fused_clusters<4>(C, p->smem_optin, p->sms), n8 = fused_clusters<8>(C, p->smem_optin, p->sms);
        const int n16 = fused_clusters<16>(C, p->smem_optin, p->sms);
        const int a = n1 < n2 ? n1 : n2, b = n4 < n8 ? n4 : n8, c = a < b ? a : b;
        p->max_clusters[C] = c < n16 ? c : n16;
    }
    if (const char* v = getenv("MOE_B200_FUSED")) moe_plan_set_knob(p, 0, MOE_KNOB_FUSED, atoi(v));
    if (const char* v = getenv("MOE_B200_CLUSTER")) moe_plan_set_knob(p, 0, MOE_KNOB_CLUSTER, atoi(v));
    if (const char* v = getenv("MOE_B200_HOST_DIRECT")) moe_plan_set_knob(p, 0, MOE_KNOB_HOST_DIRECT, atoi(v));
    if (const char* v = getenv("MOE_B200_SPLIT_UNITS")) moe_plan_set_knob(p, 0, MOE_KNOB_SPLIT_UNITS, atoi(v));
    // one CTA per SM must actually fit (Section 3.2: the launcher verifies the realised occupancy)
    const int st = p->stages_for(64, 64);
    if (st < 2 || p->stages_for(p->n_hw(p->chunk()), p->chunk()) < 2) { delete p; return fail(MOE_ERR_OCCUPANCY, "shape needs more shared memory than one SM offers"); }
    const int smem = moe::smem_layout(64, 64, top_k, E, H, I, st, false, false).total + 1024;
    const int optin = p->smem_optin;
    if (!resident<64, 64>(optin, smem) || !resident<32, 32>(optin, smem) || !resident<16, 16>(optin, smem) || !resident<32, 32, true>(optin, smem) || !resident<16, 16, true>(optin, smem) ||
        !resident<16, 8>(optin, smem) || !resident<16, 4>(optin, smem) || !resident<16, 2>(optin, smem) ||
        !resident<16, 1>(optin, smem)) {
        delete p;
        return fail(MOE_ERR_OCCUPANCY, "persistent kernel is not resident with %d bytes of shared memory", smem);
    }
    if (!get_encode_fn()) { delete p; return fail(MOE_ERR_CUDA, "driver does not export cuTensorMapEncodeTiled"); }
    *out = p;
    return MOE_OK;
}

int moe_plan(int H, int E, int I, int top_k, int scoring, int renorm, moe_plan_t* out) {
    return moe_plan_ex(H, E, I, top_k, scoring, renorm, 1.0f, out);
}

void moe_plan_destroy(moe_plan_t plan) { delete plan; }

size_t moe_workspace_bytes(moe_plan_t plan, int T_max) {
    if (!plan || T_max < 1) return 0;
    size_t need = 0;                      // the layout depends on the kernel variant: cover every T up to T_max
    for (int T = 1; T <= plan->cap(T_max); ++T) { const size_t b = plan->layout(T).total; if (b > need) need = b; }
    return need;
}

int moe_workspace_init(moe_plan_t plan, void* workspace, size_t workspace_bytes, moe_stream_t stream) {
    if (!plan) return fail(MOE_ERR_ARG, "plan is NULL");
    if (!workspace) return fail(MOE_ERR_WORKSPACE, "workspace is NULL");
    if (reinterpret_cast<uintptr_t>(workspace) & 255u) return fail(MOE_ERR_ALIGN, "workspace must be 256-byte aligned");
    const WsLayout L = plan->layout(1);
    if (workspace_bytes < L.total) return fail(MOE_ERR_WORKSPACE, "workspace too small");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (cudaMemsetAsync(workspace, 0, L.flags_end, s) != cudaSuccess)
        return fail(MOE_ERR_CUDA, "cudaMemsetAsync failed: %s", cudaGetErrorString(cudaGetLastError()));
    // Fused variants: their exchange words carry the launch tag, and the tag restarts with the control words -- so no
    // word of those regions may keep an old tag (or, in fresh memory, something that looks like one).
    for (int T = 1; T <= kFusedMaxT; ++T) {
        if (!plan->fused(T)) continue;
        const WsLayout F = plan->layout(T, true);
        if (F.total > workspace_bytes) continue;             // a workspace sized for fewer tokens: that layout is never used on it
        if (cudaMemsetAsync(static_cast<uint8_t*>(workspace) + F.ll, 0, F.total - F.ll, s) != cudaSuccess)
            return fail(MOE_ERR_CUDA, "cudaMemsetAsync failed: %s", cudaGetErrorString(cudaGetLastError()));
    }
    return MOE_OK;
}

int moe_forward(moe_plan_t plan, int T, const void* hidden_bf16, const void* Wr_bf16, const float* sel_bias,
                const void* W13_fp8, const float* W13_scale, const void* W2_fp8, const float* W2_scale,
                void* out_bf16, void* workspace, size_t workspace_bytes, moe_stream_t stream) {
    int rc = check_forward_args(plan, T, hidden_bf16, Wr_bf16, sel_bias, W13_fp8, W13_scale, W2_fp8, W2_scale, out_bf16, workspace);
    if (rc != MOE_OK) return rc;
    for (int t0 = 0; t0 < T; t0 += plan->chunk()) {
        const int tc = plan->cap(T - t0);
        rc = forward_chunk(plan, tc, static_cast<const uint16_t*>(hidden_bf16) + (size_t)t0 * plan->H, Wr_bf16, sel_bias,
                           W13_fp8, W13_scale, W2_fp8, W2_scale, static_cast<uint16_t*>(out_bf16) + (size_t)t0 * plan->H,
                           workspace, workspace_bytes, static_cast<cudaStream_t>(stream));
        if (rc != MOE_OK) return rc;
    }
    return MOE_OK;
}

// ---------------------------------------------------------------------------------------------------------------
// Entry point for callers that must not allocate: the scratch lives in a fixed array in the device image.
// ---------------------------------------------------------------------------------------------------------------
static __device__ __align__(256) unsigned char g_noalloc_scratch[MOE_NOALLOC_SCRATCH_BYTES];

namespace {
std::mutex g_noalloc_mu;
void* g_noalloc_ptr[64] = {nullptr};   // device address of g_noalloc_scratch, per device ordinal
}  // namespace

int moe_forward_noalloc(moe_plan_t plan, int T, const void* hidden_bf16, const void* Wr_bf16, const float* sel_bias,
                        const void* W13_fp8, const float* W13_scale, const void* W2_fp8, const float* W2_scale,
                        void* out_bf16, moe_stream_t stream) {
    if (!plan) return fail(MOE_ERR_ARG, "plan is NULL");
    if (T < 1 || T > 64)
        return fail(MOE_ERR_ARG, "moe_forward_noalloc handles 1..64 tokens per call (got %d)", T);
    // the fused variant where its scratch fits the array, the general kernel where only that one's does
    bool fused = plan->fused(T);
    WsLayout L = plan->layout(T, fused);
    if (fused && L.total > MOE_NOALLOC_SCRATCH_BYTES) { fused = false; L = plan->layout(T, false); }
    if (L.total > MOE_NOALLOC_SCRATCH_BYTES)
        return fail(MOE_ERR_WORKSPACE, "this shape with T=%d needs %zu bytes of scratch; the built-in array holds %u",
                    T, L.total, (unsigned)MOE_NOALLOC_SCRATCH_BYTES);
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev != plan->device || dev < 0 || dev >= 64)
        return fail(MOE_ERR_ARG, "the plan's device must be the current device");
    void* ws = nullptr;
    {
        // First call on this device: resolve the array's device address.  In host code the array's name is only a
        // handle, so the address has to come from the runtime, with the owning device current.
        std::lock_guard<std::mutex> lock(g_noalloc_mu);
        if (!g_noalloc_ptr[dev]) {
            void* ptr = nullptr;
            cudaError_t e = cudaGetSymbolAddress(&ptr, g_noalloc_scratch);
            if (e != cudaSuccess || !ptr)
                return fail(MOE_ERR_CUDA, "cudaGetSymbolAddress failed: %s", cudaGetErrorString(e));
            g_noalloc_ptr[dev] = ptr;
        }
        ws = g_noalloc_ptr[dev];
    }
    int rc = check_forward_args(plan, T, hidden_bf16, Wr_bf16, sel_bias, W13_fp8, W13_scale, W2_fp8, W2_scale, out_bf16, ws);
    if (rc != MOE_OK) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // The array keeps whatever the previous call left: start every call from cleared status, counters and flags.  The
    // launch epoch (the first word) is NOT cleared: it keeps counting across calls, which is what tells this call's
    // flags and tagged words from the ones earlier calls left in the array.
    if (cudaMemsetAsync(static_cast<uint8_t*>(ws) + 4, 0, L.flags_end - 4, s) != cudaSuccess)
        return fail(MOE_ERR_CUDA, "cudaMemsetAsync failed: %s", cudaGetErrorString(cudaGetLastError()));

    // descriptors are encoded on the stack: no descriptor cache, nothing allocated
    return run_step(plan, T, fused, L, false, hidden_bf16, Wr_bf16, sel_bias, W13_fp8, W13_scale, W2_fp8, W2_scale, out_bf16, ws, s);
}

int moe_forward_host(moe_plan_t plan, int T, const void* hidden_host, const void* Wr_bf16, const float* sel_bias,
                     const void* W13_fp8, const float* W13_scale, const void* W2_fp8, const float* W2_scale,
                     void* out_host, void* workspace, size_t workspace_bytes, moe_stream_t stream) {
    if (!plan) return fail(MOE_ERR_ARG, "plan is NULL");
    if (!hidden_host || !out_host) return fail(MOE_ERR_ARG, "a host buffer is NULL");
    if (!workspace) return fail(MOE_ERR_WORKSPACE, "workspace is NULL");
    if (T < 1) return fail(MOE_ERR_ARG, "T must be >= 1 (got %d)", T);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    uint8_t* w = static_cast<uint8_t*>(workspace);
    // Pinned (page-locked, mapped) host buffers are addressable from the device.  A few tokens' worth of output is then
    // written by the kernel straight into `out_host` (posted writes, visible to the host once the stream is
    // synchronised) instead of through a staging area and a copy-engine transfer; likewise a small `hidden_host` can be
    // read in place.  Pageable buffers, and anything larger, take the staged path.
    auto mapped = [](const void* host_ptr) -> void* {
        cudaPointerAttributes a;
        if (cudaPointerGetAttributes(&a, host_ptr) != cudaSuccess) { cudaGetLastError(); return nullptr; }
        return (a.type == cudaMemoryTypeHost && a.devicePointer && aligned16(a.devicePointer)) ? a.devicePointer : nullptr;
    };
    const size_t row_bytes = (size_t)plan->H * 2;
    void* out_dev = (plan->host_direct & 1) && (size_t)T * row_bytes <= (64u << 10) ? mapped(out_host) : nullptr;
    void* in_dev = (plan->host_direct & 2) && (size_t)T * row_bytes <= (64u << 10) ? mapped(hidden_host) : nullptr;
    for (int t0 = 0; t0 < T; t0 += plan->chunk()) {
        const int tc = plan->cap(T - t0);
        const WsLayout L = plan->layout(tc);
        if (workspace_bytes < L.total) return fail(MOE_ERR_WORKSPACE, "workspace has %zu bytes, %zu needed for T=%d", workspace_bytes, L.total, tc);
        const size_t bytes = (size_t)tc * row_bytes;
        const uint8_t* src = static_cast<const uint8_t*>(hidden_host) + (size_t)t0 * row_bytes;
        uint8_t* dst = static_cast<uint8_t*>(out_host) + (size_t)t0 * row_bytes;
        const void* k_in = in_dev ? static_cast<const void*>(static_cast<uint8_t*>(in_dev) + (size_t)t0 * row_bytes) : static_cast<const void*>(w + L.stage_in);
        void* k_out = out_dev ? static_cast<void*>(static_cast<uint8_t*>(out_dev) + (size_t)t0 * row_bytes) : static_cast<void*>(w + L.stage_out);
        if (!in_dev && cudaMemcpyAsync(w + L.stage_in, src, bytes, cudaMemcpyHostToDevice, s) != cudaSuccess)
            return fail(MOE_ERR_CUDA, "host-to-device copy failed: %s", cudaGetErrorString(cudaGetLastError()));
        int rc = check_forward_args(plan, tc, k_in, Wr_bf16, sel_bias, W13_fp8, W13_scale, W2_fp8, W2_scale, k_out, workspace);
        if (rc == MOE_OK)
            rc = forward_chunk(plan, tc, k_in, Wr_bf16, sel_bias, W13_fp8, W13_scale, W2_fp8, W2_scale, k_out,
                               workspace, workspace_bytes, s);
        if (rc != MOE_OK) return rc;
        if (!out_dev && cudaMemcpyAsync(dst, w + L.stage_out, bytes, cudaMemcpyDeviceToHost, s) != cudaSuccess)
            return fail(MOE_ERR_CUDA, "device-to-host copy failed: %s", cudaGetErrorString(cudaGetLastError()));
    }
    return MOE_OK;
}

int moe_forward_debug(moe_plan_t plan, int T, const void* hidden_bf16, const void* Wr_bf16, const float* sel_bias,
                      const void* W13_fp8, const float* W13_scale, const void* W2_fp8, const float* W2_scale,
                      void* out_bf16, void* workspace, size_t workspace_bytes, moe_stream_t stream,
                      int32_t* topk_ids, float* topk_w, uint8_t* xq, float* xs, float* logits) {
    if (plan && T > plan->chunk()) return fail(MOE_ERR_ARG, "moe_forward_debug needs T <= %d (one launch)", plan->chunk());
    int rc = moe_forward(plan, T, hidden_bf16, Wr_bf16, sel_bias, W13_fp8, W13_scale, W2_fp8, W2_scale, out_bf16, workspace,
                         workspace_bytes, stream);
    if (rc != MOE_OK) return rc;
    const WsLayout L = plan->layout(T);
    const uint8_t* w = static_cast<const uint8_t*>(workspace);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaSuccess;
    if (topk_ids && e == cudaSuccess) e = cudaMemcpyAsync(topk_ids, w + L.ids, (size_t)T * plan->K * 4, cudaMemcpyDeviceToDevice, s);
    if (topk_w && e == cudaSuccess) e = cudaMemcpyAsync(topk_w, w + L.wts, (size_t)T * plan->K * 4, cudaMemcpyDeviceToDevice, s);
    if (xq && e == cudaSuccess) e = cudaMemcpyAsync(xq, w + L.xq, (size_t)T * plan->H, cudaMemcpyDeviceToDevice, s);
    if (xs && e == cudaSuccess) e = cudaMemcpyAsync(xs, w + L.xs, (size_t)T * (plan->H / 128) * 4, cudaMemcpyDeviceToDevice, s);
    if (logits && e == cudaSuccess) e = cudaMemcpyAsync(logits, w + L.logits, (size_t)T * plan->E * 4, cudaMemcpyDeviceToDevice, s);
    if (e != cudaSuccess) return fail(MOE_ERR_CUDA, "debug copy failed: %s", cudaGetErrorString(e));
    return MOE_OK;
}

int moe_sync_status(moe_plan_t plan, void* workspace, moe_stream_t stream) {
    if (!plan) return fail(MOE_ERR_ARG, "plan is NULL");
    if (!workspace) {
        // the built-in array of moe_forward_noalloc on the plan's device (resolved by that entry point's first call)
        std::lock_guard<std::mutex> lock(g_noalloc_mu);
        workspace = (plan->device >= 0 && plan->device < 64) ? g_noalloc_ptr[plan->device] : nullptr;
        if (!workspace) return fail(MOE_ERR_ARG, "workspace is NULL and moe_forward_noalloc has not run on the plan's device");
    }
    unsigned ctrl[8] = {0};
    cudaError_t e = cudaStreamSynchronize(static_cast<cudaStream_t>(stream));
    if (e == cudaSuccess) e = cudaMemcpy(ctrl, workspace, sizeof(ctrl), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return fail(MOE_ERR_CUDA, "CUDA error while reading status: %s", cudaGetErrorString(e));
    if (ctrl[moe::kStatus] != 0 || ctrl[moe::kAbort] != 0) {
        const unsigned st = ctrl[moe::kStatus];
        return fail(MOE_ERR_TIMEOUT, "device wait ran out (site %u, CTA %u); re-initialise the workspace", (st >> 8) & 0xFF, st >> 16);
    }
    return MOE_OK;
}

int moe_debug_stamps(moe_plan_t plan, void* workspace, moe_stream_t stream, uint64_t* host_out) {
    if (!plan || !workspace || !host_out) return fail(MOE_ERR_ARG, "plan, workspace or host_out is NULL");
    const WsLayout L = plan->layout(1);
    cudaError_t e = cudaStreamSynchronize(static_cast<cudaStream_t>(stream));
    if (e == cudaSuccess)
        e = cudaMemcpy(host_out, static_cast<const uint8_t*>(workspace) + L.stamps, (size_t)plan->sms * moe::kStampsPerCta * 8, cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return fail(MOE_ERR_CUDA, "CUDA error while reading stamps: %s", cudaGetErrorString(e));
    return MOE_OK;
}

int moe_tokens_per_launch(moe_plan_t plan) { return plan ? plan->chunk() : 0; }

int moe_plan_info(moe_plan_t plan, int T, int* grid, int* stages, int* n_hw, int* smem_bytes) {
    if (!plan || T < 1) return fail(MOE_ERR_ARG, "bad arguments");
    const int Tc = plan->cap(T);
    if (plan->fused(Tc)) {
        const int st = plan->fused_stages(Tc);
        if (grid) *grid = plan->fused_grid(Tc);
        if (stages) *stages = st;
        if (n_hw) *n_hw = moe::kFusedN;
        if (smem_bytes) *smem_bytes = moe::fused_smem_layout(Plan::fused_tc(Tc), Tc, plan->K, plan->E, plan->H, st).total + 1024;
        return MOE_OK;
    }
    const int N = plan->n_hw(Tc), st = plan->stages_for(N, Tc);
    if (grid) *grid = plan->sms;
    if (stages) *stages = st;
    if (n_hw) *n_hw = N;
    if (smem_bytes) *smem_bytes = moe::smem_layout(N, Tc, plan->K, plan->E, plan->H, plan->I, st, plan->compact(Tc), plan->weighted(Tc)).total + 1024;
    return MOE_OK;
}

int moe_plan_variant(moe_plan_t plan, int T, int* fused, int* cluster) {
    if (!plan || T < 1) return fail(MOE_ERR_ARG, "bad arguments");
    const int Tc = plan->cap(T);
    const bool f = plan->fused(Tc);
    if (fused) *fused = f ? (plan->fused_dyn(Tc) ? 2 : 1) : 0;
    if (cluster) *cluster = f ? plan->fused_cluster(Tc) : 1;
    return MOE_OK;
}

int moe_plan_set_timeout_ms(moe_plan_t plan, int ms) {
    if (!plan || ms < 1) return fail(MOE_ERR_ARG, "bad arguments");
    plan->timeout_ns = (unsigned long long)ms * 1000000ull;
    return MOE_OK;
}

}  // extern "C"
