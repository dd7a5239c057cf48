/*
 * ears.h -- C ABI of the EARS speculative-decoding verification step for
 * NVIDIA B200 (sm_100a).
 *
 * One call verifies K draft tokens for each of B independent sequences
 * ("Efficient Adaptive Rejection Sampling", arXiv 2512.13194):
 *
 *   1. every target and draft logits row becomes a temperature softmax
 *      (Sec. 3.1; temperature as discussed in Sec. 4.3);
 *   2. draft token x_k is accepted iff
 *          R_k >= max(U_k - Tolerance_k, 0),
 *          R_k = P_t(x_k) / max(P_d(x_k), 1e-10),
 *          Tolerance_k = beta * (1 - max_v P_t(v))
 *      (Sec. 3.2: uncertainty, tolerance equation, acceptance condition;
 *       Sec. 3.3 item 2: division guard and threshold clamp);
 *   3. the first rejected position n ends the accepted prefix (Sec. 3.1);
 *   4. position n receives a token drawn from normalize(max(0, P_t - P_d)) of
 *      that position, or, when all K were accepted (n = K), a token drawn from
 *      P_t of the extra target row.  The paper leaves this step to the target
 *      model ("generate ... starting from position i", Sec. 3.1); the rule used
 *      is the speculative-sampling one of its refs. [1], [2].
 *
 * Random numbers (not in the paper; fixed here so results are reproducible and
 * independent of how a batch is split): Philox4x32-10 with
 *     key     = (seed[31:0], seed[63:32])
 *     counter = (offset[31:0], offset[63:32], b_global, slot)
 *   slot k in [0,K): U_k = (word0 >> 8) * 2^-24              (exact in fp32)
 *   slot K         : u   = ((word0 << 32 | word1) >> 11) * 2^-53, the uniform of
 *                    the inverse-CDF draw in step 4 (token = smallest j with
 *                    u*S < C_j, C_j the running sum of the masses, S their total).
 * A caller advances `offset` by one per verification step.
 *
 * Conventions for every entry point unless stated otherwise:
 *   - logits are row-major and contiguous: target [B, K+1, V], draft [B, K, V],
 *     fp32, bf16 (bit pattern of the upper half of an fp32) or fp16 (IEEE binary16); draft tokens [B, K]
 *     int32.  -inf logits (masked vocabulary) are legal.
 *   - pointers are DEVICE pointers owned by the caller; the library neither
 *     retains nor frees them.  Logits must be aligned to their element size.
 *     When both logits bases are 16-byte aligned and V * elem_size is a multiple
 *     of 16 the rows are fetched with bulk asynchronous copies (TMA) or 16-byte
 *     vector loads, depending on the kernel the call's shape selects; otherwise
 *     slower element-wise loads are used with identical results.
 *   - `stream` is a cudaStream_t passed as void* (NULL = default stream).  Calls
 *     enqueue work and return; they do not synchronise.
 *   - outputs: out_accept_len[b] = n in [0, K]; out_tokens[b, 0:n] = the accepted
 *     draft tokens, out_tokens[b, n] = the resampled (n < K) or bonus (n = K)
 *     token, out_tokens[b, n+1:] = -1.
 *   - a sequence whose data cannot be verified (draft token outside [0, V); a NaN
 *     or +inf logit; a row with no finite logit) gets out_accept_len[b] = -1 and
 *     out_tokens[b, :] = -1, and bit EARS_DEV_INVALID_INPUT is set in the device
 *     status; other sequences are unaffected.  Nothing traps.
 *   - the return value reports host-detectable errors only (enum below); 0 = enqueued.
 */
#ifndef EARS_H
#define EARS_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define EARS_VERSION 100

enum {
    EARS_OK = 0,
    EARS_ERR_NULL = -1,      /* a required pointer is NULL */
    EARS_ERR_SHAPE = -2,     /* B, K or V < 1; K > EARS_MAX_K; V > 2^30; sizes overflow */
    EARS_ERR_PARAM = -3,     /* temperature not finite or <= 0; beta not finite or < 0; bad dtype */
    EARS_ERR_ALIGN = -4,     /* logits not aligned to their element size; workspace not 256-byte aligned */
    EARS_ERR_WORKSPACE = -5, /* caller workspace smaller than ears_workspace_bytes() */
    EARS_ERR_CUDA = -6,      /* a CUDA runtime call failed (see ears_last_cuda_error) */
    EARS_ERR_TIMEOUT = -7    /* a bounded device-side wait gave up (reported by ears_last_device_status) */
};

enum { EARS_DTYPE_F32 = 0, EARS_DTYPE_BF16 = 1, EARS_DTYPE_F16 = 2 };

/* bits of the device status word of a call */
enum { EARS_DEV_INVALID_INPUT = 1, EARS_DEV_TIMEOUT = 2 };

#define EARS_MAX_K 64

/*
 * The verification step as listed above, fp32 logits.  Uses a library-owned
 * workspace cached per (device, stream); calls sharing a stream are ordered,
 * calls on different streams are independent.
 */
int ears_verify_f32(const float* target_logits, const float* draft_logits,
                    const int32_t* draft_tokens, int B, int K, int V,
                    float temperature, float beta, uint64_t seed, uint64_t offset,
                    int32_t* out_accept_len, int32_t* out_tokens, void* stream);

/* Same, bf16 logits (pointer to 16-bit elements). */
int ears_verify_bf16(const void* target_logits, const void* draft_logits,
                     const int32_t* draft_tokens, int B, int K, int V,
                     float temperature, float beta, uint64_t seed, uint64_t offset,
                     int32_t* out_accept_len, int32_t* out_tokens, void* stream);

/* Same, fp16 (IEEE binary16) logits. */
int ears_verify_f16(const void* target_logits, const void* draft_logits,
                    const int32_t* draft_tokens, int B, int K, int V,
                    float temperature, float beta, uint64_t seed, uint64_t offset,
                    int32_t* out_accept_len, int32_t* out_tokens, void* stream);

/* Alias of ears_verify_f32 (the element type cannot be inferred from the arguments). */
int ears_verify(const void* target_logits, const void* draft_logits,
                const int32_t* draft_tokens, int B, int K, int V,
                float temperature, float beta, uint64_t seed, uint64_t offset,
                int32_t* out_accept_len, int32_t* out_tokens, void* stream);

/*
 * General form.  Beyond the arguments above:
 *   dtype       EARS_DTYPE_F32, EARS_DTYPE_BF16 or EARS_DTYPE_F16 (IEEE binary16).
 *   b_first     global index of local sequence 0; it enters the random counter so
 *               that a batch sharded across GPUs (Sec. 3.3 item 3 treats all active
 *               sequences independently) reproduces the unsharded result.
 *   out_pt_tok, out_pd_tok, out_max_pt   [B,K] double, optional (NULL to skip):
 *               P_t(x_k), P_d(x_k) and max_v P_t(v) of Sec. 3.2 step 1, for every
 *               position (also those after the first rejection).
 *   out_class   [B,K] uint8, optional: 0 reject, 1 direct accept (R >= U),
 *               2 accept via the pardon path (Sec. 3.2 step 5).
 *   out_resid_mass [B] double, optional: total mass S the final token was drawn
 *               from (the residual mass, or ~1 for a bonus token).
 *   workspace, workspace_bytes   caller-owned device scratch of at least
 *               ears_workspace_bytes(B,K,V) bytes, 256-byte aligned, contents
 *               arbitrary; or (NULL, 0) to use the library-owned one.  With a
 *               caller workspace the call allocates nothing.  Two calls that may
 *               overlap on the GPU must not share a workspace.
 */
int ears_verify_ex(int dtype, const void* target_logits, const void* draft_logits,
                   const int32_t* draft_tokens, int B, int K, int V,
                   float temperature, float beta, uint64_t seed, uint64_t offset,
                   int64_t b_first, int32_t* out_accept_len, int32_t* out_tokens,
                   double* out_pt_tok, double* out_pd_tok, double* out_max_pt,
                   uint8_t* out_class, double* out_resid_mass,
                   void* workspace, size_t workspace_bytes, void* stream);

/*
 * ears_verify_ex with a temperature and a base tolerance per sequence.  Sec. 3.3 item 3 verifies
 * all active sequences side by side and independently, and in a serving batch each request brings
 * its own sampling temperature (Sec. 4.3 discusses its effect on the tolerance) and possibly its
 * own beta (Sec. 3.2); the paper states both as scalars.
 *   seq_temperature, seq_beta   DEVICE arrays [B] of float, either may be NULL.  Where given,
 *               sequence b uses seq_temperature[b] / seq_beta[b] and the scalar argument of the
 *               same name is ignored; where NULL the scalar applies to every sequence.
 *   A value the scalar form would refuse (temperature not finite or <= 0, beta not finite or
 *   < 0) cannot be seen by the host: it marks that one sequence invalid (out_accept_len = -1,
 *   tokens -1, EARS_DEV_INVALID_INPUT), the others are unaffected.
 *   flags       0, EARS_FLAG_STOP_AT_FIRST_REJECT and / or EARS_FLAG_ENTROPY_UNCERTAINTY (for the latter
 *               see ears_verify_entropy).  Sec. 3.1: rejecting x_i discards every later
 *               draft token.  With the flag, what lies after a sequence's first rejected position
 *               (later rows and tokens, and the extra target row unless everything was accepted)
 *               is not part of the step: it is not validated and the optional per-position
 *               outputs are not written there; lengths and tokens are the same as without the
 *               flag on valid data.  Where a cluster kernel runs (the resident kernel for short
 *               rows, the cluster-streamed kernel from four sequences per SM on; see
 *               ears_set_path) those rows are not even read -- a cluster then walks a sequence
 *               position by position -- which saves their HBM traffic at the price of a longer
 *               chain per sequence; the other streaming kernels read them anyway and ignore them.
 * Everything else is as in ears_verify_ex.
 */
#define EARS_FLAG_STOP_AT_FIRST_REJECT 1u
#define EARS_FLAG_ENTROPY_UNCERTAINTY 2u   /* see ears_verify_entropy */
#define EARS_FLAGS_ALL (EARS_FLAG_STOP_AT_FIRST_REJECT | EARS_FLAG_ENTROPY_UNCERTAINTY)
int ears_verify_var(int dtype, const void* target_logits, const void* draft_logits,
                    const int32_t* draft_tokens, int B, int K, int V,
                    float temperature, float beta,
                    const float* seq_temperature, const float* seq_beta, unsigned flags,
                    uint64_t seed, uint64_t offset,
                    int64_t b_first, int32_t* out_accept_len, int32_t* out_tokens,
                    double* out_pt_tok, double* out_pd_tok, double* out_max_pt,
                    uint8_t* out_class, double* out_resid_mass,
                    void* workspace, size_t workspace_bytes, void* stream);

/*
 * ears_verify_var with the entropy of the target distribution.  Sec. 3.2 measures the target
 * model's uncertainty at a position as 1 - max_v P_t(v); Sec. 5 (future work, item 1) names the
 * distribution's entropy as a more refined measure and gives no formula.  Here
 *     H = -sum_v P_t(v) ln P_t(v)   (nats; masked entries contribute nothing)
 * comes out of the same sweep over the target row that yields its normaliser (one more
 * multiply-add per logit), and
 *   out_entropy [B,K] double, optional (NULL to skip): H of target row k, for every position
 *               (with EARS_FLAG_STOP_AT_FIRST_REJECT: up to the first rejection);
 *   flags may include EARS_FLAG_ENTROPY_UNCERTAINTY: the tolerance of Sec. 3.2 becomes
 *               beta * H / ln V in place of beta * (1 - max P_t).  H / ln V lies in [0, 1] like
 *               the printed measure (1 for a flat row, 0 for a one-hot row or V = 1); dividing by
 *               ln V is this library's reading of "entropy as the uncertainty measure".
 * Without the flag and with out_entropy = NULL this is ears_verify_var.  Everything else
 * (arguments, outputs, errors, workspace) as there; out_entropy must be 8-byte aligned.
 */
int ears_verify_entropy(int dtype, const void* target_logits, const void* draft_logits,
                        const int32_t* draft_tokens, int B, int K, int V,
                        float temperature, float beta,
                        const float* seq_temperature, const float* seq_beta, unsigned flags,
                        uint64_t seed, uint64_t offset,
                        int64_t b_first, int32_t* out_accept_len, int32_t* out_tokens,
                        double* out_pt_tok, double* out_pd_tok, double* out_max_pt,
                        uint8_t* out_class, double* out_resid_mass, double* out_entropy,
                        void* workspace, size_t workspace_bytes, void* stream);

/*
 * The temperature -> 0 limit of the step (Sec. 1 names temperature = 0 as the deterministic
 * regime; the entry points above refuse temperature <= 0 because their arithmetic divides by it).
 * In the limit every softmax is one-hot at its row's largest logit (the smallest index among
 * equal ones), max P_t = 1, the tolerance beta (1 - max P_t) of Sec. 3.2 is zero, and for a
 * greedily drafted token R_k is 1 or 0: x_k is accepted iff it is the top token of target row k.
 * The first mismatch n ends the accepted prefix (Sec. 3.1); out_tokens[b, n] is the top token of
 * target row n (row K if all K matched).  Draft logits, beta, seed and offset play no role.
 * Outputs, invalid-sequence marking (NaN, +inf, no finite logit in ANY of the K+1 target rows; a
 * draft token outside [0, V)), workspace rules and status words are those of ears_verify_ex.
 */
int ears_verify_greedy(int dtype, const void* target_logits, const int32_t* draft_tokens,
                       int B, int K, int V, int32_t* out_accept_len, int32_t* out_tokens,
                       void* workspace, size_t workspace_bytes, void* stream);

/*
 * Verification with the VOCABULARY split across devices (tensor-parallel logits).  Device r of
 * n_shards holds the columns [v_first, v_first + Vs) of every row: target_shard [B, K+1, Vs],
 * draft_shard [B, K, Vs], row-major and contiguous; the devices' column ranges are disjoint,
 * cover [0, V) and ascend with r.  draft_tokens [B, K] (ids in [0, V)) are the same everywhere.
 * The step is the one of ears_verify_ex [Sec. 3.1-3.3] on the concatenated rows, computed in
 * three local phases with two small exchanges the CALLER performs (all-gathers of device
 * buffers, e.g. NCCL; logits never move):
 *
 *   ears_shard_stats   -> out_stats [B (2K+1)] x 4 floats per row of this device's columns:
 *                         (max m, sum of exp((l - m)/T), logit of the row's draft token if its
 *                         column lies here else 0, 1 or 0 saying which).  Rows of a sequence:
 *                         target 0..K, then draft 0..K-1.
 *   -- all-gather out_stats over devices into all_stats [n_shards][B (2K+1)][4] --
 *   ears_shard_decide  -> every device combines the statistics in device order (so decisions
 *                         are bitwise identical everywhere), applies the acceptance rule of
 *                         Sec. 3.2 per position with U_k from the counter stream of ears_verify,
 *                         writes out_accept_len [B] and the accepted prefix of out_tokens
 *                         [B, K+1] (-1 elsewhere), and out_mass [B]: the mass this device's
 *                         columns hold of the row to draw from, in units of 1/Z_t
 *                         (max(0, P_t - P_d) of the rejected position, P_t of row K after K
 *                         acceptances).  Invalid sequences (as in ears_verify, or a token whose
 *                         column no device or more than one device claimed): length -1, tokens -1.
 *   -- all-gather out_mass over devices into all_mass [n_shards][B] --
 *   ears_shard_pick    -> the device whose columns contain the point u S of the cumulative mass
 *                         (devices in order; u the final uniform of ears_verify, S the total)
 *                         writes the drawn token's id into out_tokens[b, n]; the others leave
 *                         -1 there.  An element-wise MAX of out_tokens over devices completes
 *                         the step on every device.
 *
 * All pointers are device memory.  `workspace` (256-byte aligned, at least
 * ears_shard_workspace_bytes(dtype, B, K, Vs) bytes, caller-owned) carries state from phase to
 * phase: pass the same buffer, untouched, to the three calls of one step.  Calls are enqueued
 * on `stream`; nothing synchronises.  temperature, seed, offset, b_first as in ears_verify_ex.
 * Errors: as ears_verify_ex; EARS_ERR_SHAPE also for v_first / Vs outside [0, V];
 * EARS_ERR_PARAM for n_shards outside [1, EARS_MAX_SHARDS] or shard outside [0, n_shards).
 */
#define EARS_MAX_SHARDS 64
size_t ears_shard_workspace_bytes(int dtype, int B, int K, int Vs);
int ears_shard_stats(int dtype, const void* target_shard, const void* draft_shard,
                     const int32_t* draft_tokens, int B, int K, int Vs, int V, int v_first,
                     float temperature, float* out_stats,
                     void* workspace, size_t workspace_bytes, void* stream);
int ears_shard_decide(int dtype, const void* target_shard, const void* draft_shard,
                      const int32_t* draft_tokens, int B, int K, int Vs, int V, int v_first,
                      int n_shards, const float* all_stats, float temperature, float beta,
                      uint64_t seed, uint64_t offset, int64_t b_first,
                      int32_t* out_accept_len, int32_t* out_tokens, double* out_mass,
                      void* workspace, size_t workspace_bytes, void* stream);
int ears_shard_pick(int dtype, const void* target_shard, const void* draft_shard,
                    const int32_t* draft_tokens, int B, int K, int Vs, int V, int v_first,
                    int n_shards, int shard, const float* all_stats, const double* all_mass,
                    float temperature, uint64_t seed, uint64_t offset, int64_t b_first,
                    int32_t* out_tokens, void* workspace, size_t workspace_bytes, void* stream);

/*
 * Same step with HOST buffers: copies the inputs to library-owned device staging
 * buffers, runs the step, copies out_accept_len / out_tokens back and waits for
 * completion.  All pointers are host memory (pinned memory makes the copies
 * asynchronous and faster).  Returns a host error, or EARS_ERR_TIMEOUT if a device
 * wait gave up; invalid sequences are reported in the outputs as above.
 */
int ears_verify_host(int dtype, const void* target_logits, const void* draft_logits,
                     const int32_t* draft_tokens, int B, int K, int V,
                     float temperature, float beta, uint64_t seed, uint64_t offset,
                     int64_t b_first, int32_t* out_accept_len, int32_t* out_tokens,
                     void* stream);

/*
 * Verification step for callers that must not allocate device memory.
 * (The paper has no counterpart; this is a packaging variant of ears_verify_ex.)
 *
 * Some hosts of this library cannot call cudaMalloc at the moment they verify: code
 * running while a CUDA graph is being captured on the thread, a serving loop that gave
 * all device memory to its own pool at start-up and forbids later driver allocations,
 * or a latency-critical thread that must never take the allocator's device-wide lock.
 * ears_verify_ex allocates when it is given no workspace, and a caller workspace has
 * to come from somewhere.  This entry point instead keeps its scratch in a fixed
 * array of EARS_NOALLOC_SCRATCH_BYTES that is part of the library image: every GPU
 * that loads the library holds those bytes until the process exits, whether or not
 * this function is ever called.
 *
 * Arguments and results are those of ears_verify_ex without the optional outputs and
 * without a workspace; inputs and outputs are still the caller's device buffers.
 * The function calls no cudaMalloc, cudaFree or other allocating routine (keep the
 * ears_profile_* timing hooks off around it: they create events).
 *
 *   - Shapes whose scratch need, ears_workspace_bytes(B,K,V), exceeds
 *     EARS_NOALLOC_SCRATCH_BYTES are refused with EARS_ERR_WORKSPACE before anything
 *     is enqueued (B=512, K=3, V=256000 needs about 4.2 MB).
 *   - The first call on each device looks up the array's device address (and sets the
 *     kernels' shared-memory attribute); make that first call outside any stream
 *     capture.  The device must be current, as for every other entry point.
 *   - "Allocates nothing" holds once the code a call needs is resident: the CUDA driver loads
 *     a kernel when it is first launched (one kernel per element type and per launch plan:
 *     rows that stay in shared memory, long rows, 2- or 4-byte logits), and loading
 *     allocates.  Make one warm-up call per element type and kind of shape you will use,
 *     outside any capture, before the phase in which allocation is forbidden.
 *   - All calls on a device share the one array.  It keeps the previous call's
 *     contents; the counters that must start at zero are cleared at the start of every
 *     call, on the call's stream.  Calls that can overlap on the GPU (different streams
 *     without an ordering between them, or different host threads) race on it and
 *     give wrong results: serialise them, or use ears_verify_ex with separate workspaces.
 *   - out_device_status: optional DEVICE pointer to one int32; when not NULL the call's
 *     status word (EARS_DEV_* bits, 0 = clean) is copied there on `stream` after the
 *     kernels, for the caller to read once the stream has been waited for.
 */
#define EARS_NOALLOC_SCRATCH_BYTES (8u << 20)
int ears_verify_noalloc(int dtype, const void* target_logits, const void* draft_logits,
                        const int32_t* draft_tokens, int B, int K, int V,
                        float temperature, float beta, uint64_t seed, uint64_t offset,
                        int64_t b_first, int32_t* out_accept_len, int32_t* out_tokens,
                        int32_t* out_device_status, void* stream);

/* Upper bound of the scratch bytes a call with these sizes needs (either dtype). */
size_t ears_workspace_bytes(int B, int K, int V);

/*
 * Waits for `stream`, then returns the device status of the most recent call that
 * used the library-owned workspace of (current device, stream): an OR of EARS_DEV_*
 * bits (every call starts from 0), or a negative EARS_ERR_* if the wait itself failed.
 */
int ears_last_device_status(void* stream);

/* Same for a caller-owned workspace that was passed to ears_verify_ex on `stream`. */
int ears_workspace_device_status(void* workspace, void* stream);

/*
 * How the most recent call on the library-owned workspace of (current device, stream) decided its
 * positions -- the three-way decision of Sec. 3.2 step 5 as production telemetry, counted on the
 * device by the kernels themselves (no optional output is needed for it):
 *   out_counts[0] direct acceptances (R >= U), [1] acceptances by pardon (U - Tolerance <= R < U),
 *   [2] rejections, [3] sequences marked invalid.
 * A sequence contributes the positions it really decided: its accepted prefix and, if there is
 * one, its first rejection (so [2] is the number of sequences that ended in a rejection).  Waits
 * for `stream`; out_counts is a HOST array of four words.  The greedy form counts [3] only.
 */
int ears_last_decision_counts(void* stream, uint32_t out_counts[4]);

/* Same for a caller-owned workspace that was passed to a verification call on `stream`. */
int ears_workspace_decision_counts(void* workspace, void* stream, uint32_t out_counts[4]);

/*
 * Self-test of the kernels' bounded waits (every device-side wait in this library gives up
 * after a time limit, sets EARS_DEV_TIMEOUT and lets the kernel return; nothing can hang
 * the GPU).  Launches a tiny kernel that waits limit_ms (1..2000) on a barrier no thread ever
 * completes, waits for it and returns EARS_ERR_TIMEOUT when the wait gave up as designed
 * (EARS_OK would mean the limit did not work).  The context stays usable.
 */
int ears_selftest_bounded_wait(int limit_ms, void* stream);

/*
 * Test hook for the device random stream: out[i, 0:4] = Philox4x32-10 of counter
 * ctr_key[i, 0:4] and key ctr_key[i, 4:6]; both device pointers, n >= 0.
 */
int ears_philox_device(const uint32_t* ctr_key, uint32_t* out, int n, void* stream);

/*
 * Launch-plan override for tests (0 = automatic for every field):
 *   loader 1 = bulk-copy (TMA) loader where alignment allows, 2 = element-wise loader;
 *   parts  = number of pieces each row is split into for the statistics pass (clamped
 *   to what the row allows).
 * Results never depend on the plan except through floating-point summation order.
 */
int ears_set_plan(int loader, int parts);

/*
 * Choice among the four kernels, for tests and measurements (0 = automatic for both fields):
 *   path 1 = streaming kernel with a ring of shared-memory slots filled by bulk copies (the rows of
 *            a rejected position are read a second time);
 *        3 = streaming kernel whose warps read straight from global memory (same second pass);
 *        2 = resident kernel (the two rows of a position stay in the shared memory of a
 *            thread-block cluster; every logit is read once);
 *        4 = cluster-streamed kernel (the same clusters stream their slices instead of holding
 *            them; per sequence only the rows of the first rejected position are read again, in
 *            pieces that all CTAs of the launch serve; with EARS_FLAG_STOP_AT_FIRST_REJECT nothing
 *            after a first rejection is read).
 *            Forcing path 2 or 4 on a shape it cannot take (rows that do not fit a cluster's
 *            shared memory) makes the verification calls return EARS_ERR_SHAPE.  A non-zero
 *            `parts` of ears_set_plan also selects the ring kernel.
 *   cluster = CTAs per cluster of paths 2 and 4: 1, 2, 4, 8 or 16.
 * All kernels implement the same step (Sec. 3.1-3.3); results differ only through
 * floating-point summation order.  The initial values can also come from the environment,
 * read once when the library is loaded: EARS_PATH=streaming|resident|direct|cluster-streamed (or 1..4),
 * EARS_CLUSTER=1|2|4|8|16.
 */
int ears_set_path(int path, int cluster);

/*
 * Writes a one-line description of the launch plan a verification call with these sizes
 * would use on the current device (which kernel, cluster size and slices or pieces per row,
 * how many CTAs) into the HOST buffer `out` of `out_bytes` bytes (NUL-terminated, truncated
 * if short).  Launches nothing.
 */
int ears_describe_plan(int dtype, int B, int K, int V, char* out, size_t out_bytes);

/*
 * Device timing of the kernel for benchmarks.  After ears_profile_begin(max_calls) every
 * verification call (up to max_calls) records a CUDA event on its stream right before and
 * right after its kernel; nothing synchronises.  ears_profile_end waits for the last
 * recorded event, writes the per-call kernel durations in milliseconds into the host array
 * of `capacity` floats, stores the number of calls timed in *n_calls and releases the
 * events.  Not thread-safe against concurrent verification calls.
 */
int ears_profile_begin(int max_calls);
int ears_profile_end(float* kernel_ms, int capacity, int* n_calls);

const char* ears_status_string(int status);
const char* ears_last_cuda_error(void); /* text of the last failing CUDA call on this thread, or "" */
int ears_version(void);

/* Frees every library-owned workspace and staging buffer (synchronises the devices used). */
void ears_shutdown(void);

#ifdef __cplusplus
}
#endif
#endif /* EARS_H */
