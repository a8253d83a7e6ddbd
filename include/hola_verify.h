/* hola_verify.h - C ABI of the B200 (sm_100a) library for the entropy-aware verify step of Hierarchical
 * Speculative Decoding (HSD).
 *
 * One call verifies k draft tokens for each of B sequences:
 *   1. LM-head projection of the verifier for the k+1 verify positions,  l[r,v] = sum_h hidden[r,h] * W_lm[v,h]
 *      (the "higher-fidelity verifier" f_ver of the HSD section, restricted to its output layer);
 *   2. softmax statistics and Shannon entropy per position,  H = -sum_i p_i log p_i  in nats (HSD section);
 *   3. the entropy gate  g(t) = 1[H < tau]  and Eq. (1): a gated position keeps its draft token, any other
 *      position falls back to the verifier (Algorithm 1, the HSD loop);
 *   4. the fallback itself, which the paper leaves open, is the speculative-sampling test: accept draft token x
 *      iff  u * q(x) < p(x)  (u < min(1, p/q)); the first position that is not accepted ends the run;
 *   5. one new token per sequence: from the normalised residual max(0, p - q) at the first rejected position,
 *      or from p at position k when every draft was accepted, by inverse CDF with the supplied uniform
 *      (ascending token id, first token whose cumulative mass exceeds u * total).
 *
 * Two switches select the other readings of the paper's text: gate_source (entropy of the draft row instead of the
 * verifier's softmax: the HSD section's prose ties H to the draft model's uncertainty) and fallback (a greedy verifier,
 * y = argmax p, instead of the speculative-sampling test).  A zero-initialised struct gives steps 1-5 as listed.
 *
 * All pointers in hola_verify_args are DEVICE pointers unless a field says otherwise.  Every buffer is owned by
 * the caller.  The library allocates device memory (and a few KB of pinned host memory for hola_verify_host) only
 * inside hola_create and frees it in hola_destroy.
 * No function throws, aborts or exits; each returns a hola_status.
 */
#ifndef HOLA_VERIFY_H_
#define HOLA_VERIFY_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct hola_ctx hola_ctx; /* opaque: workspace, side stream, pinned staging, device properties */

typedef enum {
  HOLA_OK = 0,
  HOLA_ERR_INVALID_ARG = 1,       /* null pointer, non-positive size, misaligned buffer */
  HOLA_ERR_UNSUPPORTED_SHAPE = 2, /* H % 8 != 0, or B / k / H / V beyond what the context was created for */
  HOLA_ERR_WORKSPACE = 3,         /* device allocation failed in hola_create */
  HOLA_ERR_CUDA = 4,              /* a CUDA runtime or driver call failed; see hola_last_cuda_error */
  HOLA_ERR_NO_DEVICE = 5,         /* no sm_100 device, or the driver lacks tensor-map support */
  HOLA_ERR_STATIC_LIMIT = 6       /* hola_lm_head_entropy_static only: more verify rows than its fixed scratch holds */
} hola_status;

typedef enum { HOLA_Q_BF16 = 0, HOLA_Q_F32 = 1 } hola_q_dtype;

/* Which distribution's entropy feeds the gate g(t) = 1[H < tau].  The HSD section's prose ties H to how
 * unsure the draft model is, yet writes it with the verifier's symbol p; both readings are available. */
typedef enum {
  HOLA_GATE_TARGET_ENTROPY = 0, /* H of the verifier's softmax at the position (default) */
  HOLA_GATE_DRAFT_ENTROPY = 1   /* H(q_j) = -sum_v q_j(v) ln q_j(v) of the draft row, q used as given */
} hola_gate_source;

/* What the "otherwise" branch of Eq. (1), y_t = f_ver(...), does where the gate is off. */
typedef enum {
  HOLA_FALLBACK_SAMPLE = 0,     /* speculative-sampling test u q(x) < p(x), residual draw at the first rejection (default) */
  HOLA_FALLBACK_GREEDY = 1      /* greedy verifier: keep x iff x = argmax_v p(v) (lowest id on ties); next_tok = argmax p_n */
} hola_fallback;

/* Storage of W_lm.  HOLA_W_INT8 is the 8-bit case of the Lo-Bi quantiser applied to the LM head (Lo-Bi Optimization
 * section; the paper leaves the quantiser's format open): int8 [V][H] plus one fp32 scale per vocabulary row,
 * W8[v][h] = w_scale[v] * q[v][h].  The weights are streamed at half the bytes, expanded exactly to bf16 on chip, and
 * the scale multiplies the fp32 accumulators.  At most 256 verify rows go into one pass over W_lm in this mode. */
typedef enum {
  HOLA_W_BF16 = 0,
  HOLA_W_INT8 = 1, /* int8 weights, bf16 activations: the weights are expanded exactly on chip (W8A16)             */
  HOLA_W8A8 = 2,   /* int8 weights AND the hidden rows quantised the same way (one fp32 scale per verify row) by the
                    * library on the fly; products on the 8-bit tensor-core kind with exact int32 accumulation:
                    * l[r][v] = w_scale[v] * h_scale[r] * sum_h q_hid[r][h] * q_w[v][h].  Needs a context. */
  HOLA_W8A16 = 3,  /* int8 weights, hidden rows kept at 16-bit width as TWO 8-bit planes made on the fly: the coarse
                    * plane of HOLA_W8A8 (scale s1) and a plane of its remainder (scale s2 = s1 / 254), so that
                    * |x16 - x| <= max|x| / 64516 per row.  Both planes go through the 8-bit tensor-core kind
                    * (twice the rows, twice the rate, half the weight bytes of bf16) and
                    * l[r][v] = w_scale[v] * (s1[r] * sum_h q1[r][h] q_w[v][h] + s2[r] * sum_h q2[r][h] q_w[v][h]).
                    * At most 256 verify rows per pass over W_lm.  Needs a context. */
  HOLA_W_MIXED = 4 /* the Lo-Bi section's mixed precision on the LM head: groups of 256 vocabulary rows stored at 4, 8 or 16
                    * bits (hola_wmix below), all expanded exactly to bf16 on chip, bf16 activations as given.  W_lm of
                    * the arguments is not read.  At most 256 verify rows per pass; H a multiple of 128. */
} hola_w_dtype;

/* The weights of HOLA_W_MIXED (args->wmix points to one of these, in HOST memory; its pointers are DEVICE pointers).
 * The paper's quantiser maps sub-blocks of a weight matrix to 4, 8 or 16 bits and leaves format and sub-block open;
 * the reading built here: a sub-block is 128 consecutive hidden channels of one vocabulary row, and widths are
 * assigned per GROUP of 256 consecutive vocabulary rows (group g = rows 256 g .. 256 g + 255, the last one ragged).
 *   16 bits: the bf16 row as it is (w_scale[v] must be 1).
 *    8 bits: int8 codes, one scale per row (hola_quantize_w8): W[v][h] = w_scale[v] * q[v][h].
 *    4 bits: codes c in [-7, 7], two per byte (even h in the low nibble, two's complement), and per sub-block b an
 *            exponent e in 0..4 (hola_quantize_w4): W[v][h] = w_scale[v] * (c[v][h] << e[v][b]), so a sub-block's scale
 *            is w_scale[v] * 2^e.
 * Rows of one width are stored compactly, in vocabulary order, in that width's buffer; group_row[g] is the index of
 * group g's first row inside the buffer of its width.  w_scale (args) is indexed by vocabulary row as usual. */
typedef struct hola_wmix {
  const void* W16;             /* bf16 [rows16][H]                                                       */
  const void* W8;              /* int8 [rows8][H]                                                        */
  const void* W4;              /* bytes [rows4][H/2], two 4-bit codes each                               */
  const uint8_t* shift4;       /* uint8 [H/128][rows4]: exponent of each 4-bit sub-block, sub-block-major */
  const uint8_t* group_width;  /* uint8 [ceil(V/256)]: 4, 8 or 16                                        */
  const int32_t* group_row;    /* int32 [ceil(V/256)]                                                    */
  int32_t rows16, rows8, rows4;/* rows in each buffer (0: that width does not occur, its pointers may be null) */
  int32_t reserved_;
} hola_wmix;

/* Bits of the device status word (OR-ed by the kernels; the caller clears it). */
#define HOLA_FLAG_BAD_TOKEN 1u   /* a draft token outside [0,V): treated as a rejection at that position    */
#define HOLA_FLAG_BAD_UNIFORM 2u /* a uniform outside [0,1): clamped into [0, 1 - 2^-24]                     */
#define HOLA_FLAG_TIMEOUT 4u     /* an on-chip wait ran out of iterations; outputs of this call are invalid  */
#define HOLA_FLAG_R_ZERO 8u      /* residual mass was zero (p <= q everywhere): token drawn from p instead   */

typedef struct {
  int32_t B; /* sequences, >= 0 */
  int32_t k; /* draft tokens per sequence, >= 0; k = 0 is a plain draw from p_0 */
  int32_t H; /* hidden size, multiple of 8 (row pitch must be a multiple of 16 bytes) */
  int32_t V; /* vocabulary size, >= 1 */
  const void* hidden;      /* bf16 [B][k+1][H], contiguous, 16-byte aligned                                   */
  const void* W_lm;        /* bf16 [V][H], contiguous, 16-byte aligned; read exactly once per call            */
  const int32_t* draft_tok;/* int32 [B][k]                                                                    */
  const void* draft_q;     /* [B][k][V] in q_dtype: the draft model's probabilities, used as given             */
  int32_t q_dtype;         /* hola_q_dtype                                                                    */
  const float* uniforms;   /* fp32 [B][k+1] in [0,1): [b][j<k] feeds accept test j, [b][k] feeds the one draw  */
  float tau;               /* entropy threshold in nats (paper: 1.5).  tau <= 0 or NaN: gate off; +inf: all on */
  int32_t* accept_len;     /* out int32 [B], 0..k: number of draft tokens kept                                */
  int32_t* next_tok;       /* out int32 [B], 0..V-1: the token that follows them                              */
  float* entropy;          /* out fp32 [B][k+1], nats, >= 0                                                    */
  float* logZ;             /* out fp32 [B][k+1], log-sum-exp of the logits                                     */
  float* logits_out;       /* out fp32 [B][k+1][V], optional (NULL: the context's own scratch is used)         */
  uint32_t* status_word;   /* in/out uint32 [1], optional: HOLA_FLAG_* bits are OR-ed in                       */
  int32_t gate_source;     /* hola_gate_source; 0 (zero-initialised struct) = target entropy                   */
  int32_t fallback;        /* hola_fallback; 0 = speculative sampling.  With GREEDY the uniforms are not read  */
  float* draft_entropy;    /* out fp32 [B][k], optional: H(q_j), written when gate_source = DRAFT_ENTROPY       */
  int32_t w_dtype;         /* hola_w_dtype; 0 = W_lm is bf16, otherwise W_lm is int8 [V][H] and H % 16 == 0     */
  int32_t reserved_;       /* must be 0                                                                        */
  const float* w_scale;    /* fp32 [V], required with an int8 W_lm (w_dtype != 0): scale of each vocabulary row  */
  const hola_wmix* wmix;   /* HOST pointer, required with w_dtype = HOLA_W_MIXED, else ignored                   */
} hola_verify_args;

/* Creates a context on `device` able to serve calls with B <= maxB, k <= maxK and exactly this H and V.
 * Allocates the workspace (hola_workspace_bytes) once and tells the runtime once how much shared memory the kernels
 * use.  One context serves one stream at a time.  The context also remembers, from call to call, the launch geometry
 * of each (B * (k+1), w_dtype) it has seen and the tensor maps of each (hidden, W_lm) pointer pair: a call that
 * repeats an earlier call's pointers and sizes does no set-up work on the host.  The library reads no environment
 * variable. */
hola_status hola_create(hola_ctx** out, int device, int maxB, int maxK, int H, int V);
hola_status hola_destroy(hola_ctx* ctx);

/* Debug and tuning switches of a context (for sweeps and tests; the defaults are what was measured best).  Results
 * do not depend on them, only speed and the copies hola_verify_host makes.  Setting one drops the remembered launch
 * geometry and tensor maps. */
typedef enum {
  HOLA_OPT_RING_SLOTS = 1,          /* shared-memory ring slots of the GEMM kernel: 0 = as many as fit, else 2..12      */
  HOLA_OPT_ROTATING_UNITS = 2,      /* 257-384 rows per pass: 1 = three MMAs on rotating 128-column accumulator units
                                     * (default), 0 = two MMAs and one accumulator buffer                              */
  HOLA_OPT_HOST_OVERLAP = 3,        /* hola_verify_host: 1 = the draft tensor travels on the context's stream while
                                     * the GEMM runs (default), 0 = every copy on the caller's stream                  */
  HOLA_OPT_HOST_ROWS_ON_DEMAND = 4, /* hola_verify_host: 1 = always send only the draft rows the step reads,
                                     * 0 = always the whole tensor, -1 = decide per call (default)                     */
  HOLA_OPT_PAIR_MMA = 6,            /* 384-row passes on rotating units: 1 = one MMA of N = 256 over two adjacent units
                                     * plus one of N = 128 per K step (default), 0 = three MMAs of N = 128             */
  HOLA_OPT_HOST_IN_PLACE = 7,       /* hola_verify_host with rows on demand: 1 = where draft_q is pinned host memory the
                                     * device can address, the accept/sample kernel reads the rows not sent ahead in
                                     * place over the bus (default), 0 = they are copied after a read-back of accept_len */
  HOLA_OPT_CONVERTER_GROUP = 8,     /* on-chip expansion (HOLA_W_INT8, HOLA_W_MIXED): converter warps that share one K
                                     * block, 1..8; groups of that many of the eight converter warps take whole blocks
                                     * in turn.  0 = the default (2)                                                  */
  HOLA_OPT_FUSED_PASSES = 9,        /* more verify rows than one pass over W_lm holds: 1 = all passes in one launch, in
                                     * which as many neighbouring CTA pairs as there are passes walk the same vocabulary
                                     * tiles together and keep in step (default), 2 = the same without keeping in
                                     * step, 0 = one launch per pass                                                 */
  HOLA_OPT_PASSES = 5               /* passes over W_lm the verify rows are split into: 0 = chosen by estimated cost
                                     * (default), else that many when the rows fit (at most 512 per pass)             */
} hola_option;
hola_status hola_set_option(hola_ctx* ctx, int option, int value);

/* Device bytes a context of these limits holds: fp32 logits scratch [B(k+1)][V], per-CTA softmax partials,
 * staging for hola_verify_host, a status word. */
size_t hola_workspace_bytes(int maxB, int maxK, int H, int V);

/* Enqueues the whole verify step (steps 1-5 above) on `cuda_stream` (a cudaStream_t; NULL = default stream).
 * Asynchronous: no synchronisation, no host read-back.  The return code covers host-detectable errors only;
 * device-detected conditions are reported through status_word and never fault.
 * Stream semantics are those of ordinary work on `cuda_stream`, with two things to know.  (1) The kernels are
 * launched with programmatic stream serialization and each lets its successor be scheduled early; the library's own
 * kernels wait for their predecessor before they touch anything it writes, and so does any ordinarily launched work.
 * The first kernel of a call waits for the kernel in front of the call before it reads its inputs, and nothing behind
 * it is scheduled before that wait has returned, so inputs written by the kernel just before the call are seen by all
 * of the call.  (The step-by-step entry points hola_accept_sample, hola_shard_accept and hola_shard_sample wait
 * before their first read of any input.)
 * Only a kernel that the CALLER launches right behind this call with programmatic stream serialization must execute
 * griddepcontrol.wait (cudaGridDependencySynchronize) before it reads this call's outputs.  (2) With the
 * draft-entropy gate one kernel runs on a stream owned by the context, forked from and joined back to `cuda_stream`
 * by events (it stays on `cuda_stream` while that stream is being captured into a graph). */
hola_status hola_verify(hola_ctx* ctx, const hola_verify_args* args, void* cuda_stream);

/* End-to-end form for callers whose per-step data lives in host memory.  Same computation as hola_verify, but
 * hidden, draft_tok, draft_q, uniforms are HOST pointers (pinned memory makes the copies asynchronous) and
 * accept_len, next_tok, entropy, logZ, status_word are HOST outputs; logits_out is ignored.  W_lm stays a
 * DEVICE pointer: weights are resident.  Copies in, runs, copies out and synchronises the stream.
 * While the target entropy gates (gate_source = 0) only the part of draft_q that Algorithm 1's verify step reads
 * crosses the bus: the k probabilities q_j(x_j) of each sequence, gathered on the host, and the one row q_n that the
 * residual draw of a sequence needs (none when all k drafts were kept or the fallback is greedy).  The first rows
 * of every sequence (as many as fit under the LM-head GEMM, at least row 0) are copied ahead on a stream owned by
 * the context while the GEMM runs; the accept lengths are read back once in the middle of the call and the rows
 * still missing follow.  Results are identical to hola_verify on the same data.  With the draft-entropy gate every
 * draft row is read, and for small draft tensors the whole copy hides under the GEMM anyway: then the whole tensor
 * is copied (on the context's stream, under the GEMM).  HOLA_OPT_HOST_ROWS_ON_DEMAND forces one or the
 * other.  The host buffers must stay valid until the call returns. */
hola_status hola_verify_host(hola_ctx* ctx, const hola_verify_args* args, void* cuda_stream);

/* Vocabulary-parallel form of the verify step: `world` ranks (normally one GPU each) hold contiguous ranges of the
 * vocabulary rows of W_lm, and of the vocabulary axis of draft_q; hidden, draft_tok, uniforms and q_j(x_j) are the
 * same on every rank.  The paper describes the step on one device; this is its natural split over several, with the
 * same results (the statistics of disjoint vocabulary ranges merge exactly, Eq. 1's entropy included; the draw of
 * Algorithm 1's fallback is an inverse-CDF search over ranges taken in rank order).  One step is three calls with two
 * small all-gathers between them, which the caller makes (NCCL, or anything else):
 *   1. hola_shard_lm_head: logits of this rank's range (scratch or logits_out), and record_out: per verify row the
 *      statistics of those logits, per draft position the logit of x_j where this rank owns x_j.
 *      -> all-gather of the records (hola_shard_record_bytes each), in rank order, into `records`.
 *   2. hola_shard_accept: merged entropy / logZ of all rows, the accept test, accept_len (identical on every rank;
 *      with the greedy fallback next_tok too, and the step ends here), and mass_out[b] = { mass of max(0, p_n - q_n),
 *      mass of p_n } of row n = accept_len inside this rank's range.
 *      -> all-gather of the masses ([B][2] doubles each) into `masses`.
 *   3. hola_shard_sample: every rank finds the range that holds the point u_k * R; that rank alone searches its
 *      range and writes the GLOBAL token index to next_tok[b], the others write -1 (a max over ranks gives the step's
 *      result).
 * In `args`, V is this rank's share (the context is created for it), W_lm / w_scale / draft_q / logits_out are the
 * rank's own parts, draft_tok holds global indices.  gate_source must be the target entropy. */
typedef struct hola_shard_args {
  int32_t world;          /* ranks the vocabulary is split over, >= 1                                        */
  int32_t rank;           /* this rank, 0 .. world-1                                                         */
  int32_t v_offset;       /* global index of this rank's first vocabulary row                                */
  int32_t V_global;       /* size of the whole vocabulary                                                    */
  const float* q_tok;     /* dev in  fp32 [B][k]: q_j(x_j), the same on every rank                           */
  void* record_out;       /* dev out, hola_shard_record_bytes(B, k) bytes, 16-byte aligned (call 1)          */
  const void* records;    /* dev in, world records in rank order, 16-byte aligned (calls 2 and 3)            */
  double* mass_out;       /* dev out fp64 [B][2] (call 2)                                                    */
  const double* masses;   /* dev in  fp64 [world][B][2] (call 3)                                             */
} hola_shard_args;
size_t hola_shard_record_bytes(int B, int k);
hola_status hola_shard_lm_head(hola_ctx* ctx, const hola_verify_args* args, const hola_shard_args* shard, void* cuda_stream);
hola_status hola_shard_accept(hola_ctx* ctx, const hola_verify_args* args, const hola_shard_args* shard, void* cuda_stream);
hola_status hola_shard_sample(hola_ctx* ctx, const hola_verify_args* args, const hola_shard_args* shard, void* cuda_stream);

/* Bytes the last hola_verify_host call on this context copied host-to-device and device-to-host. */
hola_status hola_host_traffic(const hola_ctx* ctx, unsigned long long* h2d_bytes, unsigned long long* d2h_bytes);

/* Partial entry points, the steps of the path exposed one by one (same argument struct).
 * hola_lm_head_entropy: steps 1-2 only; fills logits (logits_out or scratch), entropy, logZ.
 * hola_accept_sample:   steps 3-5 only, from fp32 logits in args->logits_out (required) and the entropy / logZ
 *                       arrays already present in args->entropy / args->logZ (inputs here).  The greedy fallback
 *                       needs the arg-max found by step 2 and is only available through hola_verify. */
hola_status hola_lm_head_entropy(hola_ctx* ctx, const hola_verify_args* args, void* cuda_stream);
hola_status hola_accept_sample(hola_ctx* ctx, const hola_verify_args* args, void* cuda_stream);

/* The paper has no counterpart of this entry point; it exists for callers that cannot allocate device memory.
 * Some hosts of this library may not call cudaMalloc at all: a serving engine that hands every byte of HBM to its
 * own pool at start-up, a plugin running inside someone else's process under a fixed memory budget, code between
 * the begin and end of a region where the allocator is locked.  Such callers cannot use hola_create, whose
 * workspace comes from cudaMalloc.  This call does steps 1-2 (LM-head projection, logZ, entropy) with no context:
 * the per-CTA softmax statistics that the GEMM kernel leaves for the final merge live in a 1.25 MiB array that is
 * part of the library image (every GPU that loads the library holds it until the process exits), and everything
 * else is the caller's: hidden, W_lm (inputs), logits_out (REQUIRED here, fp32 [B][k+1][V]), entropy, logZ
 * (outputs), all device pointers with the layouts given above; draft_*, uniforms, tau, accept_len, next_tok are
 * ignored.  W_lm must be bf16 (w_dtype = 0): the 8-bit modes need a context's workspace and are refused here.
 * status_word is honoured and is the only way to learn that an on-chip wait ran out (HOLA_FLAG_TIMEOUT: entropy and
 * logZ of that call are then invalid); without it such a call cannot be told from a good one.
 * Limit: B*(k+1) <= 512 verify rows, else HOLA_ERR_STATIC_LIMIT and nothing is launched.
 * Runs on the CURRENT device, asynchronously on cuda_stream.  It calls no cudaMalloc, cudaFree or other allocating
 * routine.  The first call on each device also looks up the array's device address and the driver's tensor-map
 * encoder; make that first call outside any stream capture.
 * All calls on one GPU share the array, and it keeps the previous call's contents: the library clears the one word
 * that must start at zero and overwrites the rest before reading it, so calls that follow each other on one stream
 * are safe, but two calls that overlap on the GPU (issued on different streams, say) race on it and give
 * wrong entropy / logZ.  Serialise them. */
hola_status hola_lm_head_entropy_static(const hola_verify_args* args, void* cuda_stream);

/* Quantises a bf16 W_lm [V][H] (device) to the HOLA_W_INT8 form, on the current device, asynchronously on the
 * stream: scale[v] = max_h |W[v][h]| / 127 (1 for an all-zero row), q = clip(rint(W / scale), -127, 127), evaluated in
 * fp32 with ties to even.  q_out is int8 [V][H], scale_out fp32 [V], both device buffers of the caller.  Allocates
 * nothing and needs no context. */
hola_status hola_quantize_w8(const void* W_bf16, int V, int H, void* q_out, float* scale_out, void* cuda_stream);

/* The 4-bit case of the same quantiser (Lo-Bi Optimization section; format as described at hola_wmix): `rows` bf16 rows
 * of H channels (H a multiple of 128) -> packed_out bytes [rows][H/2], scale_out fp32 [rows] = max|w| / 112 (1 for an
 * all-zero row), and per sub-block b the smallest exponent e in 0..4 with 7 * 2^e * scale >= max |w| over the sub-block
 * (4 if none), written to shift_out[b * shift_stride + row]; codes = clip(rint(w / (scale * 2^e)), -7, 7), every step
 * one fp32 operation, ties to even.  shift_stride is the row count of the whole exponent array (>= rows), so that a
 * range of rows can be written into a larger buffer by offsetting the three output pointers.  Current device,
 * asynchronous on the stream, allocates nothing. */
hola_status hola_quantize_w4(const void* W_bf16, int rows, int H, void* packed_out, uint8_t* shift_out, int shift_stride,
                             float* scale_out, void* cuda_stream);

/* Launch geometry chosen for a shape (for reports): vocabulary rows per tile of a CTA pair, grid size (CTAs),
 * shared-memory ring slots, verify rows per pass, passes over W_lm, kernel launches per hola_verify call. */
typedef struct {
  int32_t tile_v, grid, stages, rows_per_pass, passes, kernels_per_call;
} hola_plan_info;
hola_status hola_plan(const hola_ctx* ctx, int B, int k, hola_plan_info* out);            /* bf16 W_lm */
hola_status hola_plan_ex(const hola_ctx* ctx, int B, int k, int w_dtype, hola_plan_info* out);
/* The same for a shape alone: no context and no device (host arithmetic only), default tuning options.  num_sms is
 * the SM count the grid is cut for (148 on a B200), rows = B (k + 1) verify rows. */
hola_status hola_plan_for_shape(int num_sms, int H, int V, int rows, int w_dtype, hola_plan_info* out);

/* Per-kernel timing for reports.  Between hola_profile_begin and hola_profile_end every hola_verify call (at
 * most max_calls of them, max_calls <= 4096) records CUDA events on its stream around the LM-head GEMM launches
 * and around the accept/sample launch.  hola_profile_end synchronises the stream and returns the summed
 * durations in milliseconds and the number of calls recorded.  Creates events (no device memory). */
hola_status hola_profile_begin(hola_ctx* ctx, int max_calls);
hola_status hola_profile_end(hola_ctx* ctx, void* cuda_stream, double* lm_head_ms, double* accept_sample_ms,
                             int* calls);

/* Self-test of the bounded waits (the paper has no counterpart; it is how the library's failure path is exercised
 * without breaking anything).  Every on-chip wait of the kernels gives up after a fixed number of SM cycles, raises
 * HOLA_FLAG_TIMEOUT and makes its CTA leave in good order.  This call launches a two-CTA miniature of the GEMM
 * kernel's set-up (barriers, tensor memory of the pair) in which one thread and one warp per CTA wait, for at most
 * `limit_cycles` SM cycles (1e3 .. 2e8), on a barrier that nothing ever signals.  Afterwards *status_word has
 * HOLA_FLAG_TIMEOUT set (it is OR-ed in: clear it first), counters[0] = 128 (every thread reached the end) and
 * counters[1] = 4 (each of the four waits returned "give up"); the device stays usable.  status_word and counters
 * (uint32 [2], zeroed by the call) are device pointers.  Asynchronous on cuda_stream. */
hola_status hola_selftest_bounded_wait(hola_ctx* ctx, long long limit_cycles, uint32_t* status_word,
                                       uint32_t* counters, void* cuda_stream);

const char* hola_strerror(hola_status s);
/* Text of the last CUDA error seen by this context (empty string if none). */
const char* hola_last_cuda_error(const hola_ctx* ctx);
/* Library version, "major.minor". */
const char* hola_version(void);

#ifdef __cplusplus
}
#endif
#endif /* HOLA_VERIFY_H_ */
