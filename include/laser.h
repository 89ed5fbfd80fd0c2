/*
 * laser.h -- C ABI of the LASER routing library for NVIDIA B200 (sm_100a).
 *
 * LASER (Load- and Score-based Expert Routing) is an inference-time router for
 * Mixture-of-Experts layers.  For every token, in row order, this library computes
 *   1. the gate logits  x = h . W_g^T (+ bias)            [Introduction: gating network]
 *   2. the softmax scores s over all E experts             [The Method, Problem formulation]
 *   3. the top-k mass M_k and the test M_k >= eps_high     [The Method, Expansion rule]
 *   4. the candidate pool {s_i >= t_fix * s_max} united with the top-k, trimmed to the
 *      c best                                              [Algorithm 1; Final assignment]
 *   5. the k candidates with the smallest current load, ties by score
 *                                                          [Algorithm 1, StableSortByLoad]
 *   6. the load update L[e] += 1 for the k chosen experts, before the next token
 *   7. combine weights, the per-expert dispatch (counts, offsets, permuted pair ids) and
 *      per-device-bin load sums                            [Motivation: placement, N_g]
 *
 * General rules for every entry point
 *   - Pointers are DEVICE pointers unless the parameter is documented as host.
 *   - The caller owns every buffer; no routing state is kept between calls.
 *   - Work is enqueued on the given CUDA stream (a cudaStream_t passed as void*); the call
 *     returns without synchronising, except laser_route_host, which synchronises the stream
 *     before returning.
 *   - Return value: LASER_OK (0) or a negative status.  On a validation error nothing is
 *     launched and no output is touched.
 *   - The library reads no environment variable and keeps no routing state of its own.
 *   - Conditions only visible on the device are OR-ed into *status_word (device int32,
 *     may be NULL): LASER_DEV_LOAD_OVERFLOW, LASER_DEV_TIMEOUT.
 */
#ifndef LASER_H_
#define LASER_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
  LASER_OK = 0,
  LASER_ERR_INVALID_ARG = -1,      /* NULL where a buffer is required, or a size out of range */
  LASER_ERR_UNSUPPORTED = -2,      /* a documented but unimplemented mode */
  LASER_ERR_WORKSPACE_TOO_SMALL = -3,
  LASER_ERR_MISALIGNED = -4,       /* hidden / W_g base or row stride not 16-byte aligned */
  LASER_ERR_CUDA = -5,             /* a CUDA runtime call failed (launch error) */
  LASER_ERR_STATIC_SCRATCH = -6    /* laser_route_static: the parameters need more scratch than
                                      LASER_STATIC_SCRATCH_BYTES */
};

/* Bits in *status_word.
 * LOAD_OVERFLOW: on entry some load counter was negative or within T of 2^31-1, so it could
 *   overflow during the call.
 * TIMEOUT: the ordered selection runs in the same launch as the router and waits for the
 *   router's tiles; a wait gave up after about two seconds (it never should).  The layer is
 *   then abandoned: its remaining selection and its dispatch are skipped, so that no stage reads
 *   scratch records that were never written.
 * When either bit is set the call's results are unspecified (every access stays in bounds). */
enum { LASER_DEV_LOAD_OVERFLOW = 1, LASER_DEV_TIMEOUT = 2 };

enum { LASER_MAX_EXPERTS = 256 };

/*
 * Parameters of one routing call (host struct, read during the call only).
 *
 *   T            tokens (rows of hidden), >= 0
 *   d            hidden size, > 0, multiple of 8
 *   E            routed experts n, 1..LASER_MAX_EXPERTS
 *   k            experts activated per token, 1 <= k <= c
 *   c            trimming size of Algorithm 1, k <= c <= E
 *   eps_high     dominance cutoff; the paper's domain is (0,1).  0 gives vanilla top-k for
 *                every token, a value above 1 expands every token.
 *   t_fix        pool threshold relative to the best score; paper's domain (0,1], 0 allowed
 *                (pool = the c best).  eps_high > 1, t_fix = 0, c = E is load-only routing.
 *   trim_mode    0 = TOP (keep the c best of the pool).  1 = RANDOM (Algorithm 1's second mode):
 *                the pool, i.e. the first m = max(k, #{s_i >= t_fix * s_max}) experts of the
 *                score ranking, is sampled down to c* = min(c, m) candidates without
 *                replacement.  The paper names no generator; this library draws with
 *                Philox4x32-10, key = seed, counter = (token index, layer index in the call,
 *                block, 0), by a partial Fisher-Yates shuffle (j = i + u_i mod (m - i)), so a
 *                call is reproducible from (seed, inputs).  Not a tuned path.
 *   update_granularity  1 = the loads a token sees include every earlier token (the method's
 *                rule as this library reads it, and the default of every helper).
 *                0 or a multiple of 32 = RELAXED variant, not the rule and never chosen for
 *                the caller: the loads seen are refreshed only every G tokens (0: once per
 *                call).  It needs no iteration to stay exact to its own definition and is
 *                there to study how far coarser updates drift.  Other values:
 *                LASER_ERR_UNSUPPORTED.
 *   renormalize  1: combine weights are divided by their sum over the k chosen experts;
 *                0: raw softmax scores.
 *   n_bins       number of device bins B >= 1 (only used when bin_loads != NULL)
 *   ld_hidden, ld_w   row strides of hidden and W_g in elements (>= d, multiple of 8)
 */
typedef struct laser_params {
  int32_t T, d, E, k, c;
  float eps_high;
  float t_fix;
  int32_t trim_mode;
  int32_t update_granularity;
  int32_t renormalize;
  int32_t n_bins;
  int32_t fresh_loads; /* 0: loads and bin_loads are in/out and the call adds to them.
                          1: the call starts from empty counters (the method resets the loads at
                          the start of a batch): what loads and bin_loads hold on entry is ignored
                          and they return this call's counts.  (This word was padding before:
                          a zeroed structure keeps the old behaviour.) */
  int64_t ld_hidden, ld_w;
  uint64_t seed; /* RANDOM trimming: generator key */
} laser_params;

/* Library version, major*10000 + minor*100 + patch. */
int laser_version(void);

/* Static description of a status code.  Never NULL. */
const char* laser_strerror(int status);

/*
 * Scratch bytes one layer of laser_route needs for these parameters (the per-token candidate
 * records of stage 4 and the per-group records of the ordered selection).  p and bytes are host pointers.
 */
int laser_workspace_bytes(const laser_params* p, size_t* bytes);

/*
 * Route one MoE layer (stages 1-7 above).
 *
 *   hidden      [T, ld_hidden] bf16, row-major, 16-byte aligned
 *   w_g         [E, ld_w]      bf16, one row per expert, 16-byte aligned
 *   bias        [E] fp32 added to the logits, or NULL
 *   loads       [E] int32, in/out: L on entry, L + per-call counts on return
 *   expert_to_bin [E] int32 in [0, n_bins), or NULL for contiguous e / ceil(E / n_bins);
 *               an expert mapped outside that range is counted in no bin
 *   bin_loads   [n_bins] int32 in/out, or NULL to skip bin accounting
 *   p           host
 *   expert_ids  [T, k] int32 out.  Top-k branch: descending score.  Expanded branch:
 *               ascending (load seen by the token, score rank).
 *   weights     [T, k] fp32 out, weights[t,j] belongs to expert_ids[t,j]
 *   offsets     [E+1] int32 out, exclusive prefix of this call's per-expert counts
 *   perm        [T*k] int32 out: pair ids t*k+j grouped by expert, ascending within an expert
 *   logits_out  [T, E] fp32 out, or NULL.  Never changes a decision.
 *   status_word device int32 or NULL (bits are OR-ed in, never cleared)
 *   workspace   device scratch of at least laser_workspace_bytes(), 256-byte aligned
 */
int laser_route(const void* hidden, const void* w_g, const float* bias,
                int32_t* loads, const int32_t* expert_to_bin, int32_t* bin_loads,
                const laser_params* p,
                int32_t* expert_ids, float* weights, int32_t* offsets, int32_t* perm,
                float* logits_out, int32_t* status_word,
                void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Route n_layers independent MoE layers that share one shape in one call.  Layer l uses
 * element l of every array below; each layer has its own W_g, bias, loads and outputs, and
 * the result equals n_layers calls of laser_route.
 *
 *   hidden [n_layers, T, ld_hidden]   w_g [n_layers, E, ld_w]   bias [n_layers, E] or NULL
 *   loads [n_layers, E]               bin_loads [n_layers, n_bins] or NULL
 *   expert_to_bin [E] shared by all layers, or NULL
 *   eps_high_per_layer, t_fix_per_layer: HOST arrays [n_layers] or NULL (use p's value)
 *   expert_ids [n_layers, T, k]  weights [n_layers, T, k]  offsets [n_layers, E+1]
 *   perm [n_layers, T*k]         logits_out [n_layers, T, E] or NULL
 *   workspace: n_layers * laser_workspace_bytes() bytes
 */
int laser_route_layers(int32_t n_layers,
                       const void* hidden, const void* w_g, const float* bias,
                       int32_t* loads, const int32_t* expert_to_bin, int32_t* bin_loads,
                       const laser_params* p,
                       const float* eps_high_per_layer, const float* t_fix_per_layer,
                       int32_t* expert_ids, float* weights, int32_t* offsets, int32_t* perm,
                       float* logits_out, int32_t* status_word,
                       void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * laser_route_layers that also records CUDA events between its stages, so that a caller can
 * time the router + selection kernel (stages 1-6) and the dispatch kernels (7) separately.
 * stage_events is a HOST array of four cudaEvent_t handles (entries may be NULL),
 * recorded on cuda_stream: [0] at the start, [1] after the scratch flags have been cleared and
 * before the kernel that runs the contraction, the score epilogue and the ordered selection
 * with its load update, [2] after that kernel, [3] after the dispatch kernel (which also
 * writes the combine weights).  Small calls run their dispatch inside the first kernel: [3]
 * then follows [2] directly.
 * With more than 64 layers the stages run once per group of 64 and the events keep the last
 * group's marks.  stage_events == NULL makes this identical to laser_route_layers.
 */
int laser_route_layers_profiled(int32_t n_layers,
                                const void* hidden, const void* w_g, const float* bias,
                                int32_t* loads, const int32_t* expert_to_bin, int32_t* bin_loads,
                                const laser_params* p,
                                const float* eps_high_per_layer, const float* t_fix_per_layer,
                                int32_t* expert_ids, float* weights, int32_t* offsets,
                                int32_t* perm, float* logits_out, int32_t* status_word,
                                void* workspace, size_t workspace_bytes, void* cuda_stream,
                                void* const* stage_events);

/*
 * Device bytes laser_route_host needs in its arena for n_layers layers (inputs, outputs and
 * workspace).  p and bytes are host pointers.
 */
int laser_host_arena_bytes(int32_t n_layers, const laser_params* p, size_t* bytes);

/*
 * laser_route_layers with HOST buffers: copies the inputs to the device arena, routes,
 * copies expert_ids, weights, offsets, perm, loads and bin_loads back, and synchronises the
 * stream.  Every array argument has the layout of laser_route_layers but lives in host
 * memory (pinned memory makes the copies asynchronous); arena is device memory of at least
 * laser_host_arena_bytes(), 256-byte aligned.  loads / bin_loads are in/out on the host.
 * status_out (host int32, may be NULL) receives the device status word.
 */
int laser_route_host(int32_t n_layers,
                     const void* hidden, const void* w_g, const float* bias,
                     int32_t* loads, const int32_t* expert_to_bin, int32_t* bin_loads,
                     const laser_params* p,
                     const float* eps_high_per_layer, const float* t_fix_per_layer,
                     int32_t* expert_ids, float* weights, int32_t* offsets, int32_t* perm,
                     int32_t* status_out,
                     void* arena, size_t arena_bytes, void* cuda_stream);

/*
 * Imbalance figures of a finished call, computed on the device from its dispatch offsets
 * [Motivation: expert imbalance I_L = max_e N_e / mean_e N_e of a layer and batch, the
 * aggregate I_agg = sum_L w_L I_L, and the same on devices with N_g = sum_e A_{g,e} N_e for a
 * 0/1 placement; Evaluation, Metrics: MV, read as I_L - 1].
 *
 *   offsets       [n_layers, E+1] int32, as written by laser_route_layers
 *   expert_to_bin [E] int32 in [0, n_bins), or NULL for contiguous e / ceil(E / n_bins);
 *                 an expert mapped outside that range is counted in no bin, as in laser_route;
 *                 ignored when placement is given
 *   placement     [n_bins, E] fp32 row-major, or NULL: the general matrix A (A[g,e] >= 0, each
 *                 column summing to 1; a replicated expert splits its tokens); not checked
 *   imbalance     [n_layers] fp32 out: I_L (1 for a layer without assignments)
 *   bin_imbalance [n_layers] fp32 out, or NULL: the same over the n_bins device bins
 *   aggregate     [2] fp32 out, or NULL: I_agg and its bin-level counterpart (1 when
 *                 bin_imbalance is NULL).  The paper leaves w_L open; here w_L is the layer's
 *                 share of all assignments of the call, which is uniform for equal layers.
 * MV of a layer is imbalance[l] - 1.  All pointers are device pointers, caller-owned.
 * Limits: 1 <= n_layers <= 65535; 1 <= n_bins <= E without placement, <= 1024 with it.
 * Counts are exact; bin loads and ratios are formed in fp64 and rounded once to fp32.
 * Enqueues two small kernels on cuda_stream; returns LASER_ERR_INVALID_ARG on a bad
 * argument and LASER_ERR_CUDA if a launch fails.
 */
int laser_imbalance(int32_t n_layers, int32_t E, int32_t n_bins, const int32_t* offsets,
                    const int32_t* expert_to_bin, const float* placement, float* imbalance,
                    float* bin_imbalance, float* aggregate, void* cuda_stream);

/*
 * Gate-score statistics per layer, from fp32 logits (e.g. logits_out of laser_route_layers on
 * prefill batches) [Layer Variability in Gate Score Distributions: top-k mass M_k, Shannon
 * entropy, the regimes single-head / plateau / smooth; The Method, Parameter setting: these
 * figures guide eps_high and t_fix per layer or layer band].
 *
 *   logits  [n_layers, T, E] fp32, device
 *   stats   [n_layers, LASER_STATS_WORDS] int64 out, device; ACCUMULATED into when
 *           accumulate != 0 (several batches), else overwritten:
 *             0        tokens
 *             1        sum of M_k          in units of 2^-32 (exact)
 *             2        sum of the entropy  in units of 2^-32 (nats; each token rounded)
 *             3, 4, 5  tokens in the regimes single-head, plateau, smooth
 *             6        sum of n_near
 *             7        sum of the best score s_max, in units of 2^-32 (exact)
 *             8..71    histogram of M_k over 64 equal bins of [0, 1]; a dominance cutoff
 *                      that sends a wanted share of tokens to the top-k branch is a
 *                      quantile of it
 *   means   [n_layers, 4] fp32 out, or NULL: mean M_k, mean entropy, mean s_max, mean n_near
 *           of everything accumulated so far
 * Scores are the routing softmax bit for bit; M_k is formed as in the routing rule (k best by
 * logit descending, index ascending; fp32, left to right).  The paper names the regimes and
 * gives no criterion; the one used counts the experts comparable to the best,
 * n_near = #{i : s_i >= near_ratio * s_max} (the candidate-pool size for t_fix = near_ratio):
 * single-head if n_near = 1, plateau if 2 <= n_near <= plateau_max, else smooth.
 * Requires 1 <= k <= E <= LASER_MAX_EXPERTS, 0 <= near_ratio <= 1, plateau_max >= 1,
 * 0 <= T, n_layers in 1..65535, T * n_layers tokens below 2^30; else LASER_ERR_INVALID_ARG.
 * Enqueues a memset (unless accumulating) and up to two kernels on cuda_stream.
 */
#define LASER_STATS_WORDS 72
int laser_score_stats(int32_t n_layers, int32_t T, int32_t E, int32_t k, const float* logits,
                      float near_ratio, int32_t plateau_max, int32_t accumulate,
                      int64_t* stats, float* means, void* cuda_stream);

/* Size of the scratch array built into the library for laser_route_static (4 MiB). */
enum { LASER_STATIC_SCRATCH_BYTES = 4 * 1024 * 1024 };

/*
 * laser_route for callers that cannot allocate device memory.  (The paper has no
 * counterpart: this is a convenience of the library, not a step of the method.)
 *
 * laser_route needs a scratch buffer that its caller allocates.  Some callers have no way to
 * do that: code that runs inside another program's fixed memory pool, a service whose
 * allocator is frozen once it has started, a routine that may not call cudaMalloc because an
 * allocation would stall every stream of the process.  This entry point takes the same
 * inputs and outputs as laser_route, with the same results, but its scratch is an array of
 * LASER_STATIC_SCRATCH_BYTES bytes that is part of the library itself.  The cost: every GPU
 * on which the library is loaded gives up that much memory until the process exits.
 *
 *   - The call itself allocates and frees nothing, on the host side of CUDA or the device.
 *   - Parameters whose laser_workspace_bytes() is larger than LASER_STATIC_SCRATCH_BYTES are
 *     refused with LASER_ERR_STATIC_SCRATCH and nothing is launched.  One layer of 16384
 *     tokens with k = 6, c = 8 needs about 1.1 MiB.
 *   - The device that owns cuda_stream must be the current device.
 *   - The first call on each device looks up the array's device address (a runtime query,
 *     once per device, cached under a lock).  Make that first call outside any stream
 *     capture.
 *   - All calls on one device share the one array, and it keeps whatever the previous call
 *     left; the call clears the part that has to start at zero on the stream.  Two calls
 *     whose kernels can overlap on the GPU (different streams without an ordering between
 *     them) race on the array and give undefined results: order them.
 *
 * Arguments, return value and status_word are those of laser_route, without workspace and
 * workspace_bytes.
 */
int laser_route_static(const void* hidden, const void* w_g, const float* bias,
                       int32_t* loads, const int32_t* expert_to_bin, int32_t* bin_loads,
                       const laser_params* p,
                       int32_t* expert_ids, float* weights, int32_t* offsets, int32_t* perm,
                       float* logits_out, int32_t* status_word, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* LASER_H_ */
