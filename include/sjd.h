/*
 * sjd.h -- C ABI of the SJD / SJD++ verify-and-redraft step for NVIDIA B200 (sm_100a).
 *
 * One call of sjd_step() is one speculative Jacobi iteration's sampling and verification work for B
 * sequences with a window of W draft image tokens each, over a V-token vocabulary:
 *
 *   sampling head   merged = uncond + s (cond - uncond), y = merged / T, top-K filter, softmax over the
 *                   survivors (paper Section 3.1; K and the guidance weight s in Section 5.1)
 *   verification    accept draft x_i iff r < min(1, p_i(x_i) / q_i(x_i)), r ~ U[0,1)  (Eq. acc-sjdpp);
 *                   everything from the first failed test on is rejected (Section 4.1, Step 4)
 *   residual        the first rejected position is redrawn from max(0, p - q) / sum max(0, p - q)
 *                   (Eq. rej-sjd)
 *   redraft         later positions keep their draft when C_i = p_i(x_i)/q_i(x_i) > tau (Eq. reuse, the
 *                   SJD++ rule) and are otherwise redrawn from p_i; with SJD_FLAG_REUSE off every later
 *                   position is redrawn (plain SJD, Eq. refine-sjd)
 *
 * p_i is this call's distribution at window row i, q_i the distribution the draft was drawn from in the
 * previous iteration.  Distributions cross the ABI in sparse form: after top-K a row has at most
 * kcap = min(top_k, V) non-zero entries, stored as ascending token ids plus probabilities.
 *
 * All arithmetic runs in the library's CUDA kernels.  sjd_step() allocates nothing, frees nothing and
 * never synchronises: the caller owns every buffer, including the scratch workspace, and the call
 * returns as soon as the kernels are enqueued on params->stream.  (The host-buffer variant at the end of
 * this header owns device mirrors and does synchronise.)
 *
 * Random numbers: Philox4x32-10, key = (seed low word, seed high word), counter = (absolute position,
 * sequence index, Jacobi iteration, purpose); one block per decision, no state.  A uniform for the accept
 * test is (x0 >> 8) * 2^-24.  Sampling uses a fixed-point inverse CDF: weight w_k -> floor(w_k * 2^40),
 * T = sum, t = floor((x0 | x1 << 32) * T / 2^64), result = first entry (ascending token id) whose running
 * sum exceeds t.
 *
 * Unless stated otherwise every pointer below is a DEVICE pointer valid on the device that is current
 * when the call is made.  No entry point throws; errors are reported by the return value.
 */
#ifndef SJD_H_
#define SJD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SJD_VERSION 1
#define SJD_W_MAX 512 /* largest window of the paper's window-size ablation */
#define SJD_STATIC_MAX_ROWS 16384 /* largest B*W sjd_step_static() accepts */

/* logits_dtype */
#define SJD_F32 0
#define SJD_BF16 1
#define SJD_F16 2 /* IEEE half precision */

/* flags */
#define SJD_FLAG_REUSE 1     /* Eq. reuse (SJD++); clear = Eq. refine-sjd (SJD)                              */
#define SJD_FLAG_DRAFT_ALL 2 /* no verification: draw every valid row from its own p (initial drafts; Section
                                4.2 strategies that sample from a predicted distribution).  accept_len = 0. */

#define SJD_FLAG_NO_REFINE 16 /* sjd_window_advance() only: the "no refinement" ablation of the paper's analysis
                                section - nothing is carried over, every slot behind the committed tokens is
                                newly initialised; sjd_step() ignores it                                   */

#define SJD_FLAG_FORCE_GENERIC 4 /* diagnostics: use the any-shape multi-pass row kernel even where a
                                   single-pass kernel applies (results are identical)                    */
#define SJD_FLAG_FORCE_TILES 8   /* diagnostics: skip the single-pass kernel that cuts a row into one id
                                   range per thread; the tile-dealing one is used where it applies        */

/* cnt value of a row of sjd_probs that stands for the uniform distribution over V (1/V each); used for
 * window slots that were initialised at random and have no previous-iteration distribution. */
#define SJD_Q_UNIFORM (-1)

/* out_flags values */
#define SJD_OUT_INVALID 0   /* row >= win_len                         */
#define SJD_OUT_ACCEPTED 1  /* draft kept, part of the accepted prefix */
#define SJD_OUT_RESIDUAL 2  /* first rejected row, residual sample     */
#define SJD_OUT_REUSED 3    /* draft kept by the confidence rule       */
#define SJD_OUT_RESAMPLED 4 /* redrawn from p_i                        */

/* status bits (per sequence, OR-ed) */
#define SJD_STATUS_QTOK_NONPOSITIVE 1 /* q_i(x_i) <= 0 at a valid row: treated as an infinite ratio      */
#define SJD_STATUS_EMPTY_RESIDUAL 2   /* fixed-point residual total was 0: drawn from p instead          */
#define SJD_STATUS_DEGENERATE_ROW 4   /* a row had no finite logit: its probabilities are all 0          */
#define SJD_STATUS_INTERNAL_TIMEOUT 8 /* a bounded on-chip wait gave up: the sequence's outputs are invalid */
#define SJD_STATUS_ROW_REDONE 16      /* informational: a row did not fit the single-pass kernel's on-chip lists
                                         and was redone by the any-shape path; its result is exact, the step slower */

/* return codes */
#define SJD_OK 0
#define SJD_ERR_NULL (-1)      /* a required pointer is NULL                                              */
#define SJD_ERR_SHAPE (-2)     /* B < 0, W outside 1..SJD_W_MAX, V < 8 or not a multiple of 8, top_k < 1  */
#define SJD_ERR_ALIGN (-3)     /* logits base or strides not 16-byte aligned                              */
#define SJD_ERR_DTYPE (-4)     /* unknown logits_dtype                                                    */
#define SJD_ERR_WORKSPACE (-5) /* workspace NULL, misaligned or smaller than sjd_workspace_bytes()        */
#define SJD_ERR_STRUCT (-6)    /* params->struct_size does not match this header                          */
#define SJD_ERR_CUDA (-7)      /* a CUDA runtime call failed (see sjd_last_cuda_error)                    */
#define SJD_ERR_CAPACITY (-8)  /* a fixed-capacity entry point was given a problem beyond its limit       */

/* A set of per-position distributions plus the probability of one designated token per position.
 * Row r = b*W + i.  Rows at or beyond a sequence's win_len have cnt = 0. */
typedef struct {
  float* tok_prob; /* [B,W]       probability of the token in the matching token array (drafts / out_tokens) */
  int32_t* ids;    /* [B,W,kcap]  support of the row, ascending token id                                     */
  float* vals;     /* [B,W,kcap]  probabilities on that support                                              */
  int32_t* cnt;    /* [B,W]       entries used (kcap for a valid row), or SJD_Q_UNIFORM on input             */
} sjd_probs;

/* Token initialisation of new window slots (Section 4.2, "Token Initialization with Spatial Prior"). */
#define SJD_INIT_RANDOM 0        /* uniform token, uniform reference distribution (vanilla Jacobi decoding) */
#define SJD_INIT_REPEAT_LEFT 1   /* strategy (a): the token of the left neighbour, position p-1            */
#define SJD_INIT_REPEAT_ABOVE 2  /* strategy (b): the token of the neighbour above, position p-G           */
#define SJD_INIT_SAMPLE_LEFT 3   /* strategy (c): a draw from the prediction made for the left neighbour   */
#define SJD_INIT_SAMPLE_ABOVE 4  /* strategy (d): a draw from the prediction made for the neighbour above  */

/* HOST struct, read during the call; device pointers inside it are read by the kernels. */
typedef struct {
  int32_t struct_size;        /* sizeof(sjd_params)                                                        */
  int32_t B, W, V;            /* sequences, window rows, vocabulary                                        */
  int32_t logits_dtype;       /* SJD_F32, SJD_BF16 or SJD_F16                                              */
  int64_t stride_b, stride_w; /* element strides of BOTH logits tensors; the vocabulary axis is contiguous;
                                 stride * element size must be a multiple of 16 bytes                      */
  float cfg_scale;            /* s; unused when logits_uncond is NULL                                      */
  float inv_temperature;      /* 1/T, rounded to float by the caller; 1.0f is an exact no-op               */
  int32_t top_k;              /* K >= 1; kcap = min(K, V)                                                  */
  float reuse_tau;            /* tau of Eq. reuse (the paper uses 0.5)                                     */
  int32_t flags;              /* SJD_FLAG_*                                                                */
  int32_t iteration0;         /* Jacobi iteration index used when `iteration` is NULL                      */
  int32_t seq_base;           /* global index of sequence 0 of this call: the generator's sequence word is
                                 seq_base + b, so a batch split over calls or GPUs draws the same numbers  */
  const int32_t* win_len;     /* [B] device, valid rows per sequence (ragged windows); NULL = W            */
  const int32_t* pos_base;    /* [B] device, absolute image-token index of window row 0; NULL = 0          */
  const int32_t* iteration;   /* [B] device, per-sequence iteration index; NULL = iteration0               */
  int32_t* out_flags;         /* [B,W] device, optional SJD_OUT_* per position                             */
  int32_t* status;            /* [B] device, optional SJD_STATUS_* bits per sequence (overwritten)         */
  void* workspace;            /* device scratch, 256-byte aligned, owned by the caller                     */
  size_t workspace_bytes;     /* >= sjd_workspace_bytes(params)                                            */
  void* stream;               /* cudaStream_t the work is enqueued on (NULL = legacy default stream)       */
  void* ev_rows_begin;        /* optional cudaEvent_t recorded on `stream` just before the row stage ...   */
  void* ev_rows_end;          /* ... and just after it (tracing; NULL = not recorded)                      */
  int32_t init_mode;          /* SJD_INIT_*: how the window functions fill new slots; sjd_step ignores it  */
  int32_t grid_width;         /* G: tokens per image row of the raster grid (the "above" strategies), >= 1 */
} sjd_params;

/* Library version (the SJD_VERSION the library was compiled with). */
int sjd_version(void);

/* Static text for a return code. */
const char* sjd_status_string(int code);

/* Text of the last CUDA runtime error seen by this thread's most recent failing call ("" if none). */
const char* sjd_last_cuda_error(void);

/* Number of kernels this library has launched in this process so far (all threads, all entry points). */
uint64_t sjd_launch_count(void);

/* Scratch bytes sjd_step() needs for this shape (depends on B, W only).  0 on a NULL argument. */
size_t sjd_workspace_bytes(const sjd_params* params);

/*
 * Which row kernel sjd_step() selects for this shape and these flags (Section 3.1's sampling head has three
 * implementations that give identical results): SJD_ROWS_RANGES, SJD_ROWS_TILES or SJD_ROWS_GENERIC, or a
 * negative SJD_ERR_* for a shape, dtype or strides sjd_step() would refuse (pointers and the workspace are not
 * looked at).  Decided from the shape alone: it assumes the driver offers the tensor-map encoder the range
 * kernel needs, which every driver that runs this library's kernels does.  Launches nothing.
 */
#define SJD_ROWS_GENERIC 0 /* any shape: radix select over global memory, several passes                   */
#define SJD_ROWS_TILES 1   /* V a multiple of 2,048: one pass, tiles dealt to the filter warps             */
#define SJD_ROWS_RANGES 2  /* V a multiple of 256, kcap <= 2,048: one pass, one id range per filter thread */
int sjd_row_kernel(const sjd_params* params);

/*
 * One verify-and-redraft step (Section 4.1 Steps 3-4 on top of the Section 3.1 sampling head).
 *
 *   logits_cond    [B,W,V] device, dtype per params; row (b,i) holds the model's logits for window row i
 *   logits_uncond  same layout, or NULL for no guidance (merged = cond)
 *   drafts         [B,W] device int32, draft token x_i of every row          (ignored with DRAFT_ALL)
 *   draft_probs    HOST struct of device arrays: q_i(x_i) in tok_prob and the full previous-iteration
 *                  rows q_i in ids/vals/cnt (needed at the first rejected row)  (ignored with DRAFT_ALL)
 *   philox_seed    key of the counter-based generator
 *   out_accept_len [B] device int32: a_b = number of leading rows whose test passed, 0..win_len_b
 *   out_tokens     [B,W] device int32: row < a: the draft; row a: residual sample; a < row < win_len:
 *                  reused draft or new sample; row >= win_len: -1
 *   out_probs      HOST struct of device arrays: tok_prob = p_i(out_tokens); ids/vals/cnt = p_i of every
 *                  valid row.  After the caller shifts the window it is a valid draft_probs for the next
 *                  iteration.  Must not alias draft_probs or the logits.
 *
 * Asynchronous on params->stream.  Returns SJD_OK once the kernels are enqueued.  A negative SJD_ERR_* for a
 * bad argument means that nothing was enqueued; SJD_ERR_CUDA (a launch or an event record refused by the
 * runtime) may leave the work enqueued before the failing call on the stream.  Conditions found on the
 * device (status bits) never abort the kernels.  A problem of more than 32 rows per SM takes several launches
 * of the row kernel.
 */
int sjd_step(const void* logits_cond, const void* logits_uncond, const int32_t* drafts,
             const sjd_probs* draft_probs, const sjd_params* params, uint64_t philox_seed,
             int32_t* out_accept_len, int32_t* out_tokens, sjd_probs* out_probs);

/*
 * Window bookkeeping of the decode loop (Section 4.1: the preparation of the draft tokens in Step 1, the
 * commit of the verified tokens at the end of Step 3, the make-up of the next window at the end of Step 4;
 * random initialisation is the baseline of Section 4.2).
 *
 * sjd_window_init() fills the first window.  With SJD_INIT_RANDOM drafts[b,i] for i < win_len[b] is a token
 * drawn uniformly from [0,V) (Philox purpose 4, counter = (pos_base[b]+i, seq_base+b, iteration[b], 4), token =
 * floor(x0 V / 2^32)) and its reference distribution is SJD_Q_UNIFORM with tok_prob = 1/V; rows beyond win_len
 * get token -1.  With a spatial-prior mode, slot i copies slot i-1 ("left" modes, and "above" modes for
 * i < G) or slot i-G ("above" modes); a copied token is a deterministic draft, so its reference distribution
 * is the point mass on it (cnt 1, vals[0] = tok_prob = 1); slot 0 is random as above.  There are no
 * predictions yet, so the two sampling modes act as their repeating counterparts here.
 *
 * sjd_window_advance() takes what sjd_step() just produced (accept_len, out_tokens, out_probs) and
 *   - commits c_b tokens per sequence: the accepted prefix plus the residual draw at the first rejected row
 *     (c = a+1), or the whole window when every row was accepted (c = win_len); they are written to
 *     committed[b, pos_base[b] .. pos_base[b]+c) (committed is [B, n_total] device int32) and c to
 *     n_committed[b] when that is not NULL;
 *   - builds the next window in next_drafts / next_probs (which must not alias the step's outputs): row i takes
 *     the step's row i+c with that row's distribution as its reference when i+c < win_len, else a newly
 *     initialised token, with the iteration index of the step that just ran in the generator's counter:
 *       SJD_INIT_RANDOM        as in sjd_window_init();
 *       SJD_INIT_REPEAT_LEFT   the token at position p-1, point-mass reference;
 *       SJD_INIT_REPEAT_ABOVE  the token at position p-G (p-1 when p < G), point-mass reference.  The token at an
 *                              earlier position is the committed one before the verified window, the step's
 *                              output token inside it, and a new slot's own initial token after it;
 *       SJD_INIT_SAMPLE_LEFT   a draw from the distribution the step predicted for position p-1, or from the last
 *                              verified row's when p-1 lies behind the window (the nearest prediction to the
 *                              left); it also becomes the reference; fixed-point inverse CDF on Philox
 *                              purpose 5, counter = (p, seq_base+b, iteration, 5), R = x0 | x1 << 32;
 *       SJD_INIT_SAMPLE_ABOVE  the same from the row of position p-G, stepping a further G back while that
 *                              position lies behind the verified window; when it was verified before this step (its
 *                              distribution is gone) the committed token there with a point-mass reference;
 *                              when p < G (or the walk leaves the grid) as SJD_INIT_SAMPLE_LEFT.
 *     The paper names the strategies; the reference distributions, the fall-backs and the generator words are
 *     this library's.  With SJD_FLAG_NO_REFINE no row is carried over: all win_len slots of the next window
 *     are initialised as above, and only the committed tokens of this step count as known tokens;
 *   - updates win_len, pos_base, iteration in place: pos_base += c, win_len = min(W, n_total - pos_base),
 *     iteration += 1.  A sequence is finished when its win_len is 0.
 * params supplies B, W, V, top_k, seq_base, init_mode, grid_width and stream; its win_len/pos_base/iteration fields are not used
 * (the arrays are passed explicitly because they are written).  All pointers are device pointers.  Both
 * calls are asynchronous on params->stream and return SJD_OK or a negative SJD_ERR_*.
 */
int sjd_window_init(const sjd_params* params, int32_t n_total, uint64_t philox_seed, int32_t* win_len, int32_t* pos_base,
                    int32_t* iteration, int32_t* drafts, sjd_probs* draft_probs);
int sjd_window_advance(const sjd_params* params, int32_t n_total, uint64_t philox_seed, const int32_t* accept_len,
                       const int32_t* step_tokens, const sjd_probs* step_probs, int32_t* win_len, int32_t* pos_base,
                       int32_t* iteration, int32_t* next_drafts, sjd_probs* next_probs, int32_t* committed,
                       int32_t* n_committed);

/*
 * sjd_step() for callers that cannot hand over a workspace.  (The paper has no counterpart: this is a
 * convenience of this library, not a step of the method.)
 *
 * Some hosts of this library may not allocate device memory at the point where they call it: a plugin
 * that runs inside another framework's stream callback or inside a memory pool it does not own, a
 * serving loop that has frozen its allocator after start-up, a process whose device memory is handed out
 * by a supervisor.  For them the scratch of the step (one 16-byte record per window row) lives in a
 * fixed array inside the library's device image, SJD_STATIC_MAX_ROWS records long (256 KiB; every GPU that
 * loads the library holds it until the process exits).  Arguments, results and error codes are those of
 * sjd_step(), except that params->workspace and params->workspace_bytes are ignored and that
 * B * W > SJD_STATIC_MAX_ROWS is refused with SJD_ERR_CAPACITY, nothing enqueued.  The call itself never
 * calls cudaMalloc, cudaFree or any allocating routine.
 *
 * The first call on each device looks up the array's device address (cudaGetSymbolAddress, with that
 * device current) and remembers it; make that first call outside any stream capture.
 *
 * All calls on a device share the one array.  Nothing in it has to start at zero (the row stage writes
 * every record before the verification stage reads it), and it keeps the last call's contents.  Two calls
 * whose kernels can overlap on the GPU (different streams without an ordering between them) race on it:
 * order them, or use sjd_step() with separate workspaces.
 */
int sjd_step_static(const void* logits_cond, const void* logits_uncond, const int32_t* drafts,
                    const sjd_probs* draft_probs, const sjd_params* params, uint64_t philox_seed,
                    int32_t* out_accept_len, int32_t* out_tokens, sjd_probs* out_probs);

/*
 * Host-buffer variant for callers whose logits and window state live in host memory.
 *
 * sjd_host_ctx_create() allocates, on the current device, device copies of every argument of sjd_step()
 * for the shape in `shape` (B, W, V, logits_dtype, top_k are read; strides are taken as contiguous
 * [B,W,V]) plus the workspace and a stream, and returns an opaque handle.  sjd_step_host() copies the
 * HOST arrays in (pinned memory makes the copies asynchronous and fast, pageable memory works), runs
 * sjd_step() on the context's stream, copies every output back and returns after the stream has
 * drained, so the host arrays are ready on return.  In `params`, B/W/V/dtype/top_k must equal the
 * context's; win_len, pos_base, iteration, out_flags and status are HOST pointers here (or NULL);
 * workspace, stream and the event fields are ignored.  draft_probs / out_probs hold HOST pointers.
 * Returns SJD_OK or a negative SJD_ERR_*.  sjd_host_ctx_destroy() frees everything (NULL is allowed).
 * A context must not be used by two threads at once.
 */
typedef struct sjd_host_ctx sjd_host_ctx;
int sjd_host_ctx_create(const sjd_params* shape, sjd_host_ctx** out_ctx);
int sjd_step_host(sjd_host_ctx* ctx, const void* logits_cond, const void* logits_uncond, const int32_t* drafts,
                  const sjd_probs* draft_probs, const sjd_params* params, uint64_t philox_seed,
                  int32_t* out_accept_len, int32_t* out_tokens, sjd_probs* out_probs);
void sjd_host_ctx_destroy(sjd_host_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* SJD_H_ */
