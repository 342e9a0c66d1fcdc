/*
 * moe_b200.h -- C ABI of the fused routed-MoE decode step for NVIDIA B200 (sm_100a).
 *
 * One call to moe_forward() runs one decode step of the complete routed
 * Mixture-of-Experts operator of the paper (Section 3: top-k/quantize,
 * up-projection, down-projection, reduce) in ONE persistent kernel launch:
 *
 *   router logits (Section 3.3) -> softmax or sigmoid(+selection bias) top-k
 *   (Section 4.1) -> per-token 1x128 FP8 E4M3 quantisation of the input
 *   (Section 4.1) -> gate/up projection against FP8 weights with 128x128 fp32
 *   block scales, tokens on the MMA N dimension (Eq. 9) -> SiLU(gate)*up and
 *   FP8 requantisation (Section 3.3, up-projection epilogue) -> down
 *   projection -> top-k weighted reduction in fixed slot order (Section 3.2).
 *
 * Conventions
 *   - All tensor pointers are DEVICE pointers, row-major, contiguous, owned by
 *     the caller; the library never frees or reallocates them.  Every pointer
 *     must be 16-byte aligned.
 *   - H and I must be multiples of 128, 1 <= top_k <= min(E, 32), E <= 512.
 *   - W13 rows [0,I) of each expert are the gate projection, rows [I,2I) the
 *     up projection.
 *   - Calls are asynchronous on `stream`; nothing synchronises the host.
 *   - Every function returns MOE_OK or a negative error code and never throws
 *     or aborts; moe_last_error() returns a description of the most recent
 *     failure on the calling thread.  Problems found on the device (a wait that
 *     ran out) are recorded in the workspace and read with moe_sync_status().
 *   - There is no CPU fallback: without a CUDA device of compute capability
 *     10.x every entry point that needs one returns MOE_ERR_UNSUPPORTED_ARCH.
 */
#ifndef MOE_B200_H_
#define MOE_B200_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct moe_plan* moe_plan_t;
typedef void* moe_stream_t; /* a cudaStream_t */

enum {
    MOE_OK = 0,
    MOE_ERR_ARG = -1,              /* null pointer, T out of range, ... */
    MOE_ERR_SHAPE = -2,            /* H/I not multiples of 128, top_k or E out of range */
    MOE_ERR_ALIGN = -3,            /* a pointer is not 16-byte aligned */
    MOE_ERR_WORKSPACE = -4,        /* workspace missing or too small */
    MOE_ERR_CUDA = -5,             /* a CUDA runtime/driver call failed */
    MOE_ERR_OCCUPANCY = -6,        /* the persistent grid cannot be co-resident */
    MOE_ERR_TIMEOUT = -7,          /* a device-side wait ran out (see moe_sync_status) */
    MOE_ERR_UNSUPPORTED_ARCH = -8  /* no sm_100 device */
};

enum { MOE_SCORE_SOFTMAX = 0, MOE_SCORE_SIGMOID_BIAS = 1 };

/* Largest number of tokens one kernel launch can handle; a plan's own limit is moe_tokens_per_launch(). */
#define MOE_MAX_TOKENS_PER_LAUNCH 128

/* Size of the scratch array built into the library's device image for moe_forward_noalloc (24 MiB). */
#define MOE_NOALLOC_SCRATCH_BYTES (24u << 20)

/*
 * moe_plan: fix the layer shape and routing policy (Section 3.4: shape and
 * schedule are fixed ahead of time, token count is a run-time argument).
 *   H hidden size, E experts, I intermediate size, top_k experts per token,
 *   scoring MOE_SCORE_*, renorm != 0 renormalises the selected weights.
 * Queries the current device, checks that the persistent grid (one CTA per SM)
 * is actually co-resident, one CTA per SM, rather than assuming it (Section
 * 3.2), and stores host-side state only.  *out receives the plan; free it with moe_plan_destroy.
 */
int moe_plan(int H, int E, int I, int top_k, int scoring, int renorm, moe_plan_t* out);

/* As moe_plan, plus the routed scaling factor multiplied into the routing weights (Section 4.1: 2.5 for the
 * sigmoid policies; 1.0 otherwise). */
int moe_plan_ex(int H, int E, int I, int top_k, int scoring, int renorm, float routed_scale, moe_plan_t* out);

void moe_plan_destroy(moe_plan_t plan);

/* Bytes of device scratch a call with up to T_max tokens needs (flags, logits, quantised activations,
 * intermediate FP8 tile, split-K partials, per-slot outputs).  0 on invalid arguments. */
size_t moe_workspace_bytes(moe_plan_t plan, int T_max);

/* Zero the control words and flags of a workspace.  Must run once (stream-ordered) before the first
 * moe_forward that uses the workspace, and again after an MOE_ERR_TIMEOUT.  `workspace` is device memory,
 * 256-byte aligned, of at least moe_workspace_bytes() bytes. */
int moe_workspace_init(moe_plan_t plan, void* workspace, size_t workspace_bytes, moe_stream_t stream);

/*
 * moe_forward: one decode step for T tokens (Section 3; Eq. 9 for the projections).
 *   hidden_bf16 [T,H] bf16          Wr_bf16 [E,H] bf16         sel_bias [E] fp32 or NULL (sigmoid policy only)
 *   W13_fp8 [E,2I,H] E4M3 bytes     W13_scale [E,2I/128,H/128] fp32
 *   W2_fp8  [E,H,I]  E4M3 bytes     W2_scale  [E,H/128,I/128] fp32
 *   out_bf16 [T,H] bf16 (written)   workspace: see moe_workspace_init; sized for >= min(T, moe_tokens_per_launch()) tokens
 * All launches that share one workspace must be ordered on the device (same stream, or events): two calls
 * that overlap on the GPU race on the scratch.  More tokens than moe_tokens_per_launch() are processed as
 * consecutive launches of at most that many tokens.
 * Returns MOE_OK once the work is enqueued.
 */
int moe_forward(moe_plan_t plan, int T,
                const void* hidden_bf16, const void* Wr_bf16, const float* sel_bias,
                const void* W13_fp8, const float* W13_scale,
                const void* W2_fp8, const float* W2_scale,
                void* out_bf16, void* workspace, size_t workspace_bytes, moe_stream_t stream);

/*
 * moe_forward_host: moe_forward with the step's activations in HOST memory (Section 3: same operator).
 *   hidden_host [T,H] bf16 and out_host [T,H] bf16 are host pointers (pinned memory makes the copies asynchronous);
 *   every other tensor is a device pointer as in moe_forward.  Enqueues, on `stream`: a host-to-device copy of
 *   `hidden_host` into a staging area of the workspace, the kernel, and a device-to-host copy of the result; with
 *   pinned buffers of at most 64 KiB the kernel writes the result into `out_host` itself (see MOE_KNOB_HOST_DIRECT).
 *   The host buffers must stay valid, and `out_host` must not be read, until the stream has been synchronised.
 */
int moe_forward_host(moe_plan_t plan, int T,
                     const void* hidden_host, const void* Wr_bf16, const float* sel_bias,
                     const void* W13_fp8, const float* W13_scale,
                     const void* W2_fp8, const float* W2_scale,
                     void* out_host, void* workspace, size_t workspace_bytes, moe_stream_t stream);

/*
 * moe_forward_noalloc: moe_forward for callers that cannot give the library device memory.  (The paper has no
 * counterpart: this entry point exists only for integration.)  Some hosts of this library may not call cudaMalloc
 * at the point where they run a decode step -- for instance code running inside a memory pool that owns the whole
 * device, or a runtime whose allocator is not reentrant from the thread that launches kernels -- and so they have
 * no scratch buffer to hand over.  Here the scratch is a fixed array of MOE_NOALLOC_SCRATCH_BYTES (24 MiB) that is
 * part of the library's device image: every GPU that loads the library holds these 24 MiB until the process exits.
 *   - Same tensor arguments as moe_forward; there is no workspace argument.  1 <= T <= 64.
 *   - A layer shape whose scratch for T tokens exceeds the array is rejected with MOE_ERR_WORKSPACE and a message
 *     giving both sizes (the five benchmark shapes fit for T <= 16).  Up to 8 tokens the fused-unit kernel variant
 *     is used where its (larger) scratch fits, the general variant otherwise; results agree within rounding.
 *   - A device-side wait that ran out is recorded in the array, like in a workspace: read it with
 *     moe_sync_status(plan, NULL, stream) BEFORE the next moe_forward_noalloc call on the device (every call starts by
 *     clearing the array's control words, and with them the record).
 *   - The plan's device must be the current device.  The FIRST call on a device looks up the array's device
 *     address (cudaGetSymbolAddress); make that first call outside any stream capture.
 *   - The call itself allocates nothing: no cudaMalloc/cudaFree, no descriptor cache; TMA descriptors are built on
 *     the stack.  It enqueues one small memset (control words and flags, which must start from zero because the
 *     array keeps the previous call's contents) and the kernel, both on `stream`.
 *   - All calls on a device share the one array: calls that overlap on the GPU (different streams without an
 *     ordering between them, or different host threads) race.  Order them.
 */
int moe_forward_noalloc(moe_plan_t plan, int T,
                        const void* hidden_bf16, const void* Wr_bf16, const float* sel_bias,
                        const void* W13_fp8, const float* W13_scale,
                        const void* W2_fp8, const float* W2_scale,
                        void* out_bf16, moe_stream_t stream);

/*
 * moe_forward_debug: moe_forward, then copies (device to device, on `stream`) the routing and input
 * quantisation results of the step into caller buffers; any of them may be NULL.  Requires
 * T <= moe_tokens_per_launch().
 *   topk_ids [T,top_k] int32 (slot order: key descending, index ascending)   topk_w [T,top_k] fp32
 *   xq [T,H] E4M3 bytes   xs [T,H/128] fp32   logits [T,E] fp32
 */
int moe_forward_debug(moe_plan_t plan, int T,
                      const void* hidden_bf16, const void* Wr_bf16, const float* sel_bias,
                      const void* W13_fp8, const float* W13_scale,
                      const void* W2_fp8, const float* W2_scale,
                      void* out_bf16, void* workspace, size_t workspace_bytes, moe_stream_t stream,
                      int32_t* topk_ids, float* topk_w, uint8_t* xq, float* xs, float* logits);

/* Synchronise `stream`, read the workspace's device status word and return MOE_OK, MOE_ERR_TIMEOUT or
 * MOE_ERR_CUDA.  After MOE_ERR_TIMEOUT the workspace must be re-initialised.  workspace == NULL reads the built-in
 * array of moe_forward_noalloc on the plan's device (MOE_ERR_ARG if that entry point has never run there). */
int moe_sync_status(moe_plan_t plan, void* workspace, moe_stream_t stream);

/* Tokens one launch of this plan handles: 128 when the routing is sparse enough (128 * top_k <= 20 * E) for the
 * kernel to compact each expert's tokens into its MMA columns (Eq. 9 puts tokens on the N dimension), otherwise 64. */
int moe_tokens_per_launch(moe_plan_t plan);

/* Introspection: persistent grid size, pipeline stages and hardware N used for T tokens; any out may be NULL. */
int moe_plan_info(moe_plan_t plan, int T, int* grid, int* stages, int* n_hw, int* smem_bytes);

/* Introspection: which kernel variant T tokens get.  *fused = 1 or 2 for the fused-unit variant (1..16 tokens: a work
 * unit is one expert's 128-wide intermediate block through gate/up AND its down-projection column block, shared by
 * the *cluster CTAs of a thread-block cluster; Section 3.2's hand-over of the intermediate tile stays on chip), 0 for
 * the general variant (*cluster = 1).  2: the launch is made in pairs (*cluster = 2) and the kernel decides after
 * routing whether the CTAs of a pair share units (the step has at most as many units as pairs) or work alone.
 * Either out may be NULL. */
int moe_plan_variant(moe_plan_t plan, int T, int* fused, int* cluster);

/* Diagnostics: synchronise `stream` and copy the phase time stamps of the last launch on this workspace to
 * HOST memory host_out[SMs*32] (nanoseconds of the GPU's global timer; 32 words per CTA, the first 16 in use); the launch must have run with MOE_KNOB_STAMPS
 * set.  Fused-unit variant, per CTA: 0 start, 1 router rows published, 2 input quantised, 3 all logits gathered, 4 top-k
 * done, 5 routing metadata done, 6 first weight tile requested, 7 first weight tile landed, 8 first accumulator read,
 * 9 first partial sums parked, 10 first intermediate tile ready, 11 last down tile stored, 12 all CTAs done, 13
 * reduction done, 14 SM id (not a time), 15 exit.  General variant, per CTA: 0 start, 1 input quantised,
 * 2 router logits done, 3 arrived at the routing flag, 4 routing published grid-wide, 5 selection keys ready,
 * 6 top-k done, 7 routing metadata done, 8 first weight tile requested, 9 first ring of requests issued,
 * 10 first weight tile landed, 11 first accumulator read, 12 up phase done, 13 down phase done, 14 reduction
 * done, 15 exit.  Section 3.3 of the paper argues which of these gaps must hide under the weight stream. */
int moe_debug_stamps(moe_plan_t plan, void* workspace, moe_stream_t stream, uint64_t* host_out);

/*
 * Schedule knobs (Section 3.4: shape and schedule are fixed ahead of time; the paper finds its schedule with an
 * offline search, and so does paper_2609_04244_b200/tune.py through these two calls).  T = 0 sets a per-token-count
 * knob for every token count; COMPACT_MIN and PDL are plan-wide and ignore T.  Changing MOE_KNOB_COMPACT_MIN changes
 * which kernel variant a token count gets and with it the scratch layout: query moe_workspace_bytes() again.
 *   MOE_KNOB_STAGES            pipeline stages of the shared-memory ring, 2..16 (capped by what fits); 0 = the
 *                              library's choice for the token count (default): 6 or 8 for short weight streams, all
 *                              that fit for steps of a few tiles and for long streams
 *   MOE_KNOB_SPLIT_SLACK_KIB   keep a projection's units whole while that costs the busiest CTA at most this many KiB
 *                              of extra weight stream, split them across CTAs (split-K) otherwise (default 200 up to 8 tokens,
 *                              100 beyond)
 *   MOE_KNOB_ROUTE_ALL_TOKENS  up to this many tokens every CTA selects the experts of all tokens; beyond, the grid
 *                              shares the tokens and exchanges the result (default 8; up to 8 tokens every CTA always
 *                              selects for all of them, so smaller values act as 8)
 *   MOE_KNOB_COMPACT_MIN       fewest tokens (2..9) for which each expert's tokens are compacted into its MMA columns (9)
 *   MOE_KNOB_PDL               programmatic dependent launch on/off (1)
 *   MOE_KNOB_SPLIT_WEIGHT      where tokens are compacted: cut the k-step lists into per-CTA ranges of equal WEIGHT, a
 *                              k-step of an expert with many tokens weighing more (its epilogue work grows with the
 *                              columns in use), instead of ranges of equal length.  0 = equal length, 1..8 = strength
 *                              of the per-column term in quarters of the fitted value, -1 = the library's choice
 *                              (default: 4 from 24 tokens on, from 16 where I <= 256, else 0)
 *   MOE_KNOB_FUSED             (per token count 1..16) kernel variant: 1 = the fused-unit variant if it can run, 0 = the
 *                              general variant, -1 = the library's choice (default).  Changes the scratch layout: query
 *                              moe_workspace_bytes() again.
 *   MOE_KNOB_CLUSTER           fused-unit variant: CTAs that share one unit (thread-block cluster size) 1, 2, 4 or 8;
 *                              0 = the library's choice (default): the size for which the busiest CTA streams the fewest
 *                              tiles at the expected number of distinct experts.  MOE_ERR_OCCUPANCY if the device cannot
 *                              hold such clusters.  With MOE_KNOB_STAGES = 0 the fused variant takes as many stages as
 *                              fit one CTA per SM.
 *   MOE_KNOB_SPLIT_UNITS       (plan-wide) fused-unit variant: 1 (default) = where a step has more units than clusters, the
 *                              list of all accumulation groups is cut into equal ranges, one per cluster; a range may begin
 *                              and end anywhere inside a unit (clusters that share a unit exchange partial sums); 2 = the
 *                              same also where the step has fewer units than clusters (ranges shorter than a unit; measured
 *                              slower than whole units on every benchmark shape, kept for experiments); 0 = units are always
 *                              dealt to clusters whole, round-robin
 *   MOE_KNOB_HOST_DIRECT       (plan-wide) moe_forward_host with PINNED host buffers of at most 64 KiB: bit 0 (default on) = the
 *                              kernel writes the result straight into out_host, bit 1 = it reads hidden_host in place; the
 *                              transfers that are not taken this way go through a staging area and the copy engine
 *   MOE_KNOB_STAMPS            (plan-wide) the fused-unit variant records the phase time stamps moe_debug_stamps() reads
 *                              (1; 2 = also inside its routing phase); off by default.  The general variant always records
 *                              its sixteen stamps: one store per phase, and guarding them measured slower
 *   MOE_KNOB_DEBUG_SKIP        (plan-wide, for tests of the give-up paths) 1: the fused-unit variant never signals that an
 *                              intermediate tile is ready, so every wait behind that signal runs out after the plan's time
 *                              limit and the launch ends with MOE_ERR_TIMEOUT -- no fault, nothing waits for ever.  0 (default)
 * Results do not depend on STAGES, ROUTE_ALL_TOKENS, PDL or STAMPS; SPLIT_SLACK_KIB, COMPACT_MIN, SPLIT_WEIGHT, FUSED and
 * CLUSTER change the order of fp32 partial sums (never the routing or the quantised input).
 */
enum { MOE_KNOB_STAGES = 0, MOE_KNOB_SPLIT_SLACK_KIB = 1, MOE_KNOB_ROUTE_ALL_TOKENS = 2, MOE_KNOB_COMPACT_MIN = 3, MOE_KNOB_PDL = 4,
       MOE_KNOB_SPLIT_WEIGHT = 5, MOE_KNOB_FUSED = 6, MOE_KNOB_CLUSTER = 7, MOE_KNOB_STAMPS = 8, MOE_KNOB_DEBUG_SKIP = 9, MOE_KNOB_SPLIT_UNITS = 10, MOE_KNOB_HOST_DIRECT = 11 };
int moe_plan_set_knob(moe_plan_t plan, int T, int knob, int value);
int moe_plan_get_knob(moe_plan_t plan, int T, int knob, int* value);

/* Set the device-side wait limit in milliseconds (default 1000).  A wait that runs out makes the kernel
 * record MOE_ERR_TIMEOUT and return; it never traps. */
int moe_plan_set_timeout_ms(moe_plan_t plan, int ms);

const char* moe_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* MOE_B200_H_ */
