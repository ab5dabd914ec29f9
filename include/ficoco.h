/*
 * libficoco -- the FiCoCo token-reduction step (filter, correlate, compress, compact)
 * as CUDA kernels for sm_100a behind a C ABI.
 *
 * What one call computes, per image (or per sequence), following the paper
 * "Filter, Correlate, Compress: Training-Free Token Reduction for MLLM Acceleration":
 *
 *   filter    Eq. 1:  s_i = lambda * (1/N) sum_j A_ij - (1 - lambda) * a_i, followed by the
 *             local penalty (2x2 windows on the patch grid, window maximum times 2; Sec.
 *             "Redundancy-based Token Discard") and a top-N^S selection of the tokens to
 *             discard (set S); the rest is the target set T.
 *   correlate Sec. "Correlation-based Information Recycling": C_ij = A_ij for i in S,
 *             j in T; tau_i = eps-quantile of row i; J_i = { j : C_ij >= tau_i }.
 *   compress  Eq. 2:  X_j <- (X_j + sum_{i in I_j} alpha_ij X_i) / (1 + sum_{i in I_j} alpha_ij),
 *             alpha_ij = C_ij / sum_{j in J_i} C_ij.
 *   compact   Algorithm 1, last step: the rows of S are removed, order preserved.
 *
 * The token-to-token relation A_ij between two vision tokens is the cosine similarity of
 * the token features; the attention-derived term a_i is supplied by the caller (CLS->patch
 * attention per head for FiCoCo-V, text->vision attention per head for FiCoCo-L) and is
 * averaged over heads.  FiCoCo-L (Sec. "Task-Aware Improvements for FiCoCo-L") uses
 * s_i = beta * v_i - (1 - beta) * (1/M) sum_k t_ki, no local penalty, and
 * C_ij = gamma * A_ij + (1 - gamma) * (1/M) sum_k t_ki t_kj with t the head-mean
 * text->vision attention.
 *
 * General rules
 *   - "device" pointers are CUDA device memory on the context's device; "host" pointers
 *     are ordinary host memory read during the call.
 *   - The caller owns every input and output buffer.  A context owns only scratch memory.
 *   - ficoco_v_reduce / ficoco_l_reduce enqueue work on the given stream and return without
 *     synchronising.  A context must be used from one stream at a time.
 *   - The first call with a new combination of shapes builds and uploads a small plan
 *     (per-image descriptors); that first call may synchronise the stream and must happen
 *     outside stream capture (or be replaced by ficoco_v_plan).  Up to 16 plans are cached per
 *     context.  The per-image sizes come from host arrays (seqlens, keep, grids): the library
 *     sizes its grids from them without reading anything back from the device.
 *   - Every function returns FICOCO_OK (0) or a negative ficoco_error; nothing is launched
 *     when argument validation fails.  Problems only the device can see (a `pos` entry
 *     outside the grid) set bits in a status word read by ficoco_status.
 *   - No output buffer may overlap an input buffer of the same call (Eq. 2 reads the tokens
 *     as they were before the update); such a call returns FICOCO_ERR_INVALID_ARG.
 *   - Device-side waits (between the thread blocks of one kernel) are bounded by elapsed time.
 *     Should one run out, the step stops writing, bit 2 of the status word is raised, and every
 *     later step of the context does nothing until ficoco_status has read and cleared it.
 *   - Token rows must be 16-byte aligned: dim % 8 == 0 for bf16, dim % 4 == 0 for fp32.
 *     A token row of all zeros has no direction; its cosine is taken as 0.
 *   - At most 8192 vision tokens per image; the top list needed for tau_i,
 *     n - floor(eps * (n - 1)) entries for n preserved tokens, must not exceed 16.
 */
#ifndef FICOCO_H_
#define FICOCO_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct ficoco_ctx ficoco_ctx;

enum ficoco_dtype { FICOCO_FP32 = 0, FICOCO_BF16 = 1 };

enum ficoco_error {
  FICOCO_OK = 0,
  FICOCO_ERR_INVALID_ARG = -1,   /* NULL pointer, non-positive size, misaligned pointer */
  FICOCO_ERR_UNSUPPORTED = -2,   /* dtype / dim / per-image size / quantile level outside the supported range */
  FICOCO_ERR_KEEP_RANGE = -3,    /* keep count < 0 or > number of alive vision tokens */
  FICOCO_ERR_WORKSPACE = -4,     /* problem larger than the sizes given to ficoco_create */
  FICOCO_ERR_CUDA = -5,          /* a CUDA runtime call failed (see ficoco_last_cuda_error) */
  FICOCO_ERR_TIMEOUT = -6,       /* a bounded device-side wait ran out */
  FICOCO_ERR_CAPTURE = -7,       /* a new plan would have to be uploaded during stream capture */
  FICOCO_ERR_GRID = -8,          /* grid_h * grid_w smaller than the number of alive patches */
  FICOCO_ERR_STATIC_LIMIT = -9   /* problem larger than the fixed scratch of the allocation-free entry point */
};

enum ficoco_flags {
  FICOCO_HAS_CLS = 1u,           /* row 0 of every image is a CLS token: never scored, always kept */
  FICOCO_LOCAL_PENALTY = 2u,     /* apply the local penalty (FiCoCo-V default) */
  FICOCO_AVERAGE_COMPRESSION = 4u, /* ablation "average compression" (Sec. "Ablation Study", Compress:
                                    the features are averaged directly): every alpha_ij of Eq. 2
                                    is 1, so a preserved token becomes the plain mean of itself
                                    and the discarded tokens sent to it; J_i is unchanged */
  FICOCO_CONVERGENT = 16u,       /* ablation "convergent correlation" (Sec. "Correlation-based Information
                                    Recycling" and the ablation tables: all discarded tokens merge into one
                                    additional token).  The paper gives no weights: the additional token is
                                    the plain mean of the image's discarded tokens.  Preserved tokens stay as
                                    they are; an image that discards at least one token gets one more output
                                    row right after its preserved vision rows (before the text rows of
                                    FiCoCo-L), with kept_idx -1; out_tokens and kept_idx must have room for
                                    it.  max_targets and eps are ignored. */
  FICOCO_BACK_TO_BACK = 8u       /* scheduling hint, no effect on results: the caller states that the
                                    work enqueued on the stream right before this call is the
                                    previous reduce step of this library (any context) and nothing
                                    else.  The step's first kernel may then start reading tokens
                                    and attention while that previous step is still finishing,
                                    provided its inputs do not overlap that step's outputs (the
                                    library checks the address ranges).  Without the flag every
                                    step starts in plain stream order, which is what a stream
                                    that also carries other kernels needs. */
};

/* Hyper-parameters; defaults are the paper's (Sec. "Implementation Details"):
 * lambda 0.35, beta 0.6, gamma 0.6, eps 0.998, penalty coefficient 2, window 2. */
typedef struct ficoco_params {
  double lambda_;       /* Eq. 1 balance (FiCoCo-V) */
  double beta;          /* score balance (FiCoCo-L) */
  double gamma;         /* direct / text-bridged balance in C^l (FiCoCo-L) */
  double eps;           /* quantile level of the token-wise threshold tau_i, in [0, 1] */
  double penalty_coef;  /* local-penalty scaling coefficient */
  int window;           /* local-penalty window side, >= 1 */
  int max_targets;      /* < 0: token-adaptive K (the paper's method); 0: pruning only;
                           k > 0: every discarded token goes to its k most correlated targets */
  unsigned flags;       /* ficoco_flags */
  int reserved;
} ficoco_params;

/* Fill *p with the paper's defaults and flags = HAS_CLS | LOCAL_PENALTY. */
void ficoco_default_params(ficoco_params* p);

/* Create a context on `device` with scratch sized for
 *   max_tokens : upper bound on the total number of token rows in one call (all images),
 *   max_dim    : upper bound on the hidden size,
 *   max_batch  : upper bound on the number of images / sequences per call,
 *   max_text   : upper bound on text tokens per sequence (0 if ficoco_l_reduce is not used).
 * Allocates device memory once; no later device-pointer call allocates.  *out receives the
 * context. */
int ficoco_create(ficoco_ctx** out, int device, long long max_tokens, int max_dim,
                  int max_batch, int max_text);
int ficoco_destroy(ficoco_ctx* ctx);

const char* ficoco_strerror(int code);
/* The CUDA error code behind the last FICOCO_ERR_CUDA of this context (0 if none). */
int ficoco_last_cuda_error(const ficoco_ctx* ctx);

/*
 * FiCoCo-V reduce step (Algorithm 1) for a batch of images.
 *
 * Packing.  Image b has c (0 or 1, from FICOCO_HAS_CLS) CLS rows followed by Np_b alive
 * patch rows.  Uniform batches give n_tokens = c + Np for all images; ragged batches give
 * `seqlens` (host, B entries, each c + Np_b) and n_tokens is ignored.  In both cases rows
 * are packed back to back: image b starts at row sum_{b'<b} (c + Np_b').
 * Per-patch arrays (pos, scores_out) are packed the same way without the CLS rows.
 * attn holds, per image, an [H, Np_b] row-major block; blocks are back to back, so image b
 * starts at float offset H * sum_{b'<b} Np_b' (for a uniform batch this is [B, H, Np]).
 */
typedef struct ficoco_v_args {
  const void* tokens;      /* device, dtype elements, [rows, dim] row-major */
  const int* seqlens;      /* host int32[B] rows per image incl. CLS, or NULL for uniform */
  const float* attn;       /* device fp32, CLS->patch attention weights per head */
  const int* grid_h;       /* host int32[n_grid]: rows of the original patch grid */
  const int* grid_w;       /* host int32[n_grid]: columns of the original patch grid */
  const int* pos;          /* device int32 per patch: linear index r * grid_w + c on the
                              original grid (used by the local penalty); NULL means
                              pos = 0..Np-1 (nothing discarded yet) */
  const int* keep;         /* host int32[n_keep]: N^T, patch tokens preserved per image */
  void* out_tokens;        /* device, dtype, packed [sum_b (c + keep_b), dim] */
  int* kept_idx;           /* device int32, packed like out_tokens rows: for every output
                              row the row index inside its image's input (CLS = 0) */
  int* pos_out;            /* device int32 packed [sum_b keep_b]: pos of the preserved
                              patches (input to the next step), or NULL */
  float* scores_out;       /* device fp32 packed per patch: redundancy score after the
                              local penalty, or NULL */
  int dtype;               /* ficoco_dtype */
  int batch;               /* B >= 1 */
  int n_tokens;            /* rows per image incl. CLS (uniform batches) */
  int dim;                 /* D */
  int heads;               /* H >= 1 */
  int n_grid;              /* 1 (same grid for all images) or B */
  int n_keep;              /* 1 or B */
  int reserved;
  int* out_cu_seqlens;     /* device int32[B + 1] or NULL: receives the first output row of every
                              image and, last, the total number of output rows (the cu_seqlens of
                              the packed output, for the layers behind) */
} ficoco_v_args;

int ficoco_v_reduce(ficoco_ctx* ctx, const ficoco_v_args* args, const ficoco_params* params,
                    void* cuda_stream);

/* Build and upload the plan for the shapes of `args` (batch, n_tokens or seqlens, dim, heads,
 * dtype, grids, keep counts) and the settings of `params` ahead of time.  Only the host arrays of
 * `args` are read; its device pointers may be NULL.  This call may synchronise the stream and must
 * happen outside stream capture; afterwards ficoco_v_reduce with the same shapes and settings
 * neither synchronises nor fails under capture (16 plans are cached per context, least recently
 * used first out). */
int ficoco_v_plan(ficoco_ctx* ctx, const ficoco_v_args* args, const ficoco_params* params, void* cuda_stream);

/* FiCoCo-V reduce step on a caller-supplied relation matrix: the paper's own formulation, in
 * which every token-token quantity is read from the self-attention map A^v (Sec.
 * "Redundancy-based Token Discard", Eq. 1 first term; Sec. "Correlation-based Information
 * Recycling", C = A^v) instead of from the cosine similarity of the hidden states.
 *   relation  : device fp32, 4-byte aligned; image b's [Np_b, Np_b] block (row = query token,
 *               column = key token, alive patch tokens only, no CLS row or column) starts at
 *               sum_{b' < b} Np_b'^2 floats.  Read only; the caller keeps ownership.
 *   by_column : 0: v_i = (1/Np) sum_j A[i, j], Eq. 1 as printed (a constant for a row-stochastic
 *               softmax map); non-zero: v_i = (1/Np) sum_j A[j, i], the attention token i receives,
 *               as the prose of that paragraph puts it.
 * C_ij = A[S_i, T_j]; tau_i, J_i, alpha_ij, Eq. 2, the local penalty, the selection and every
 * other argument, output and error are those of ficoco_v_reduce; the tokens only feed Eq. 2.
 * The step runs unfused kernels (score, select, correlate, merge) and never reads the N x N block
 * more than twice (all of it for the scores, the rows of S for C).  Asynchronous on the stream,
 * allocates nothing. */
int ficoco_v_reduce_relation(ficoco_ctx* ctx, const ficoco_v_args* args, const float* relation,
                             int by_column, const ficoco_params* params, void* cuda_stream);

/*
 * A progressive FiCoCo-V schedule in one call: the reduce step applied n_steps times, every step
 * on the output of the one before (the paper reduces at successive encoder layers, Sec.
 * "Implementation Details"; between two steps the host model would run its layers, so this entry
 * point is the reduction part of such a schedule on its own, as the multi-step workloads use it).
 *   first     : the arguments of step 0 (tokens, pos, grid, dtype, batch, n_tokens, dim, heads) and
 *               the buffers of the LAST step's results: out_tokens [B, c + keep[n_steps-1], dim],
 *               kept_idx (row indices into the ORIGINAL input of step 0, the chain of the steps
 *               composed), pos_out [B, keep[n_steps-1]].  first->attn, first->keep and
 *               first->scores_out are ignored; batches must be uniform (seqlens NULL).
 *   n_steps   : 1 .. 8.
 *   keep      : host int32[n_steps], patch tokens preserved by each step (the same for every
 *               image), non-increasing.
 *   attn      : host array of n_steps device pointers; attn[s] holds step s's CLS->patch weights
 *               [B, H, Np_s] over the patch tokens alive at that step (Np_0 = n_tokens - c,
 *               Np_s = keep[s-1]).
 * Intermediate tokens, kept indices and positions live in the context; they are allocated (and
 * grown) by the first call that needs them, which synchronises and must therefore happen outside
 * stream capture; later calls of the same or a smaller size allocate nothing.  Every step but the
 * first is launched while the step before is still finishing and reads its input only once that
 * step is complete.  Errors and the status word are those of ficoco_v_reduce.
 */
int ficoco_v_reduce_schedule(ficoco_ctx* ctx, const ficoco_v_args* first, int n_steps, const int* keep,
                             const float* const* attn, const ficoco_params* params, void* cuda_stream);

/*
 * FiCoCo-L reduce step (Algorithm 2) for a batch of decoder sequences of equal shape.
 * Each sequence has n_vision vision rows followed by n_text text rows.  Vision rows are
 * reduced to `keep`; text rows pass through unchanged after them.
 */
typedef struct ficoco_l_args {
  const void* tokens;      /* device, [B, n_vision + n_text, dim] */
  const float* attn_t2v;   /* device fp32 [B, H, M, N]: attention of text row k to vision token i */
  const int* keep;         /* host int32[n_keep]: vision tokens preserved */
  void* out_tokens;        /* device, packed [sum_b (keep_b + M), dim] */
  int* kept_idx;           /* device int32 packed like out_tokens rows (text rows: N..N+M-1) */
  float* scores_out;       /* device fp32 [B, N] redundancy score s^l, or NULL */
  int dtype;
  int batch;
  int n_vision;            /* N */
  int n_text;              /* M >= 1 */
  int dim;
  int heads;
  int n_keep;              /* 1 or B */
  int reserved;
} ficoco_l_args;

int ficoco_l_reduce(ficoco_ctx* ctx, const ficoco_l_args* args, const ficoco_params* params,
                    void* cuda_stream);

/*
 * Host-buffer variants: every pointer of the args struct that is documented "device" is a
 * HOST pointer here.  The call copies the inputs to the device, runs the same kernels,
 * copies the outputs back and returns after the results are in host memory.  Staging
 * buffers are allocated inside the context on the first host call (sized by the maxima
 * given to ficoco_create) and reused.  Large batches go through in groups of images (V) or
 * sequences (L) whose uploads, kernels and downloads overlap on three internal streams; the
 * results are the same bytes as those of one device-buffer call on the whole batch.
 */
int ficoco_v_reduce_host(ficoco_ctx* ctx, const ficoco_v_args* host_args,
                         const ficoco_params* params);
int ficoco_l_reduce_host(ficoco_ctx* ctx, const ficoco_l_args* host_args,
                         const ficoco_params* params);

/* Synchronise `cuda_stream`, read and clear the device status word into *device_status
 * (0 = clean; bit 0 (1): a pos entry outside grid_h*grid_w was ignored by the local penalty;
 * bit 2 (4): a bounded device-side wait ran out: the outputs of that step and of every step
 * enqueued after it are invalid; bit 3 (8): an internal index list held a token index outside
 * its image, which was replaced by 0 instead of being followed: the outputs of that step are
 * invalid).  Returns FICOCO_OK when the word could be read, whatever it holds. */
int ficoco_status(ficoco_ctx* ctx, void* cuda_stream, int* device_status);

/* Testing hook for the bounded waits.  wait_ns > 0 sets the time after which a device-side wait
 * of this context gives up (default 20 ms); extra_arrivals > 0 makes the fused filter kernel wait
 * for that many arrivals more than will ever come, so that the wait runs out by itself (nothing
 * spins past the bound, nothing faults); 0 restores normal operation.  Affects later calls. */
int ficoco_debug_waits(ficoco_ctx* ctx, long long wait_ns, int extra_arrivals);

/*
 * Inspection of the intermediate results of the most recent reduce call on this context
 * (for tests and debugging).  Synchronises the device, then copies up to `bytes` bytes of
 * the selected array to `host_dst`; *bytes_avail (optional) receives the array's size.
 * Arrays are packed over images in call order.
 */
enum ficoco_inspect_what {
  FICOCO_INSPECT_RNORM = 0,      /* fp32 per patch: 1 / ||x_i|| */
  FICOCO_INSPECT_SCORE_RAW = 1,  /* fp32 per patch: score before the local penalty */
  FICOCO_INSPECT_SCORE = 2,      /* fp32 per patch: score after the local penalty */
  FICOCO_INSPECT_SRC_IDX = 3,    /* int32 per discarded token: patch index, ascending */
  FICOCO_INSPECT_TGT_IDX = 4,    /* int32 per preserved token: patch index, ascending */
  FICOCO_INSPECT_CORR_CNT = 5,   /* int32 per discarded token: |J_i| */
  FICOCO_INSPECT_CORR_TGT = 6,   /* int32 [discarded, 16]: positions in T of the targets */
  FICOCO_INSPECT_CORR_W = 7,     /* fp32  [discarded, 16]: alpha_ij */
  FICOCO_INSPECT_CORR_C = 8,     /* fp32  [discarded, 16]: C_ij of the top list, descending */
  FICOCO_INSPECT_TAU = 9         /* fp32 per discarded token: tau_i */
};
int ficoco_inspect(ficoco_ctx* ctx, int what, void* host_dst, size_t bytes, size_t* bytes_avail);

/* Number of kernels the most recent reduce call launched (for launch accounting). */
int ficoco_last_launch_count(const ficoco_ctx* ctx);

/*
 * Per-kernel timing.  ficoco_profile(ctx, 1) clears the accumulators and makes every later
 * reduce call record a CUDA event in front of each kernel it launches (on the call's stream)
 * and one after the last; ficoco_profile(ctx, 0) stops that.  Do not enable it during stream
 * capture.  ficoco_profile_read synchronises the device, folds the recorded intervals into
 * per-kernel totals and returns entry `index` (kernels in first-launch order): its name
 * (NUL-terminated, at most name_cap bytes), the summed milliseconds and the launch count.
 * It returns FICOCO_ERR_INVALID_ARG once `index` is past the last entry.
 */
int ficoco_profile(ficoco_ctx* ctx, int enable);
int ficoco_profile_read(ficoco_ctx* ctx, int index, char* name, int name_cap, double* total_ms,
                        long long* launches);

/*
 * Equivalent token for encoders without a CLS token (appendix "Implementation of the Equivalent
 * Token"): M = mean of the key states over the heads, mu = mean of M over the image's patch
 * tokens, a_i = -cos(mu, M_i) for every patch token i.  The result stands in for the CLS
 * attention of Eq. 1: pass it to ficoco_v_reduce as `attn` with heads = 1.
 *
 * keys: device, token-major [rows, heads, head_dim] (the layout a key projection writes: one
 * contiguous row of heads * head_dim elements per token), fp32 or bf16, images packed one after
 * the other like `tokens`; a row must be a multiple of 16 bytes.  seqlens: host int32[batch]
 * rows per image (CLS row included when has_cls != 0), or NULL when every image has n_tokens
 * rows.  a_eq: device fp32, one value per patch token, packed in the same order (CLS rows left
 * out).  A patch key or a mean of zero length gives 0.
 * One thread-block cluster of 8 CTAs works on an image and keeps the head-mean keys of its
 * tokens in shared memory: an eighth of the image's patch tokens times 4 * head_dim bytes, plus
 * two staging buffers of 8 key rows, must fit in 220 KB (about 5000 patch tokens per image at
 * 16 heads of 64 bf16); a longer image, head_dim > 256 or odd, or a ragged batch of more than
 * 256 images returns FICOCO_ERR_UNSUPPORTED.  Nothing is allocated and no context is needed;
 * work is enqueued on cuda_stream and the call does not synchronise.  Should a bounded
 * device-side wait run out, the affected tokens read NaN.
 */
int ficoco_equivalent_token(const void* keys, int dtype, int batch, int n_tokens, const int* seqlens,
                            int heads, int head_dim, int has_cls, float* a_eq, void* cuda_stream);

/*
 * Allocation-free vision-aware redundancy.  (The paper has no counterpart to this entry
 * point: it exists for callers of this library that are not allowed to allocate.)
 *
 * For a uniform batch it writes, for every patch token, v_i = (1/Np) sum_j cos(x_i, x_j) over
 * the alive patches of its image (j = i included): the first term of Eq. 1, the same numbers
 * ficoco_v_reduce produces as scores when lambda = 1 and the local penalty is off.
 *
 * It needs no context and calls neither cudaMalloc nor cudaFree nor anything else that
 * allocates.  It is meant for code that runs where device allocation is off limits, typically
 * the per-step callback of a serving engine that gave all device memory to its own pool at
 * start-up: there a cudaMalloc can fail, and it synchronises the whole device.  Its scratch
 * (inverse norms and column-sum partials, about 4.7 MB) is a fixed array inside the library,
 * held by every GPU that loads the library until the process exits.  Hence:
 *   - limits: batch <= FICOCO_NOALLOC_MAX_BATCH, dim <= FICOCO_NOALLOC_MAX_DIM,
 *     batch * Np <= FICOCO_NOALLOC_MAX_ROWS; anything larger returns FICOCO_ERR_STATIC_LIMIT
 *     and launches nothing;
 *   - all calls on one device share the array and it keeps the previous call's contents;
 *     every word a call reads it has written itself first, so nothing needs clearing, but two
 *     calls that overlap on the GPU (different streams, no ordering) race on it;
 *   - the first call on each device looks up the array's device address; make that first call
 *     outside any stream capture (a first call under capture returns FICOCO_ERR_CAPTURE and
 *     launches nothing).
 * The device that owns `tokens`, `v_out` and `cuda_stream` must be the calling thread's
 * current device.  tokens: device, [batch, n_tokens, dim] (n_tokens includes the CLS row when
 * flags has FICOCO_HAS_CLS), 16-byte aligned rows; v_out: device fp32 [batch, Np].  Work is
 * enqueued on cuda_stream; the call does not synchronise.
 */
#define FICOCO_NOALLOC_MAX_ROWS 32768
#define FICOCO_NOALLOC_MAX_BATCH 64
#define FICOCO_NOALLOC_MAX_DIM 2048
int ficoco_vision_redundancy_noalloc(const void* tokens, int dtype, int batch, int n_tokens, int dim,
                                     unsigned flags, float* v_out, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* FICOCO_H_ */
