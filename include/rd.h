/*
 * rd.h -- C ABI of the recurrent-depth sampler library for NVIDIA B200 (sm_100a).
 *
 * The calls follow the paper's statement of the problem:
 *   model       e = P(x), s_0 ~ N(0, sigma^2 I), s_i = R(e, s_{i-1}), p = C(s_r)   (Section 3.1)
 *   KV sharing  one K/V entry per (layer, position), overwritten by the latest pass (Section 3.2)
 *   prefill     all prompt positions iterate the recurrence together             (Section 3.3)
 *   AR step     the sequential recurrence, one token per call                    (Section 3.1)
 *   DF step     one step of the diffusion-forcing sampler: Algorithm 1 (fixed exit) and
 *               Algorithm 2 with the exit rule of Eq. 3 (adaptive exit), wavefront limiter of
 *               Section 3.5
 *
 * Conventions
 *   - Every call returns RD_OK (0) or a negative RD_E_* code; nothing throws or aborts across
 *     this boundary; out-parameters are written only on success.
 *   - The library owns all device memory it allocates.  The caller owns every buffer it passes;
 *     buffers are borrowed for the duration of the call only (prompts and weights are copied).
 *   - "host pointer" / "device pointer" is stated per argument.  Weight pointers may be either
 *     (copied with cudaMemcpyDefault).
 *   - Steps are enqueued asynchronously on the session's stream; the calls that read results
 *     (rd_committed, rd_get_tokens, rd_debug_read, rd_stats) synchronise that stream first.
 *   - A session is used by one host thread at a time.  One session lives on one GPU: the device
 *     current when rd_load / rd_session_create are called.
 *   - All matrices are [out_features, in_features], row-major.
 */
#ifndef RD_H_
#define RD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum { RD_F32 = 0, RD_BF16 = 1 };

enum {
    RD_OK = 0,
    RD_E_INVALID_ARG = -1, /* null pointer, shape the kernels do not support, bad index      */
    RD_E_STATE = -2,       /* call out of order (step before prefill, AR inside an open wave) */
    RD_E_CAPACITY = -3,    /* prompt + budget exceed max_context, window exceeds max_window   */
    RD_E_OOM = -4,         /* device allocation failed                                        */
    RD_E_CUDA = -5,        /* a CUDA call or kernel launch failed; see rd_last_cuda_error     */
    RD_E_TIMEOUT = -6      /* a bounded device-side wait ran out (pipeline barrier)           */
};

typedef struct rd_model rd_model;     /* opaque: device weights                          */
typedef struct rd_session rd_session; /* opaque: KV caches, latents, tokens, wavefront   */

/* Model shape.  hidden must equal n_heads * head_dim and be at most 12288; hidden and mlp_inner must
 * be multiples of 8, head_dim even and <= 128.  dtype selects the storage type of weights, KV cache and GEMM
 * inputs (accumulation, residual stream, latents, softmax and logits are always float32). */
typedef struct {
    int32_t hidden, n_heads, head_dim, mlp_inner;
    int32_t n_prelude, n_core, n_coda, vocab;
    int32_t dtype;          /* RD_F32 | RD_BF16 */
    int32_t tie_embeddings; /* non-zero: the LM head is the embedding matrix */
    float rope_base;        /* rotary base (10000) */
    float norm_eps;         /* RMSNorm epsilon, added to the mean square */
    float init_sigma;       /* sigma of s_0 ~ N(0, sigma^2 I) */
} rd_config;

typedef struct {
    int32_t batch;             /* independent sequences stepped together                     */
    int32_t max_context;       /* positions per sequence the KV caches hold                  */
    int32_t max_window;        /* wavefront limiter: most in-flight positions per sequence   */
    int32_t max_iters_per_pos; /* adaptive mode: core iterations after which a position is
                                  treated as converged                                       */
    int32_t max_new_tokens;    /* N of Algorithms 1-2, per sequence                          */
    int32_t keep_logits;       /* non-zero: full logits of the last step stay readable       */
    float temperature;         /* 0 => greedy (arg max, lowest index on ties); else Gumbel-max
                                  sampling from softmax(logits / temperature)                */
    uint64_t seed;             /* key of the counter-based generator (initial states, Gumbel, noise) */
    float eta;                 /* Section 3.4: momentum on the input conditioning of rd_df_step,
                                  e = eta e_prev + (1 - eta) P(y_current) from a position's second
                                  step on; 0 <= eta < 1, 0 = off                                  */
    float beta;                /* Section 3.4 / the stabiliser steps of Algorithm 1: latent noise in rd_df_step,
                                  z <- (1 - b_t) z + b_t z_noise, b_t = beta max(0, 1 - t / T) at a
                                  position's step t; T = window (fixed exit) or
                                  ceil(max_iters_per_pos / inner_iters); 0 <= beta <= 1, 0 = off  */
    float top_p;               /* Appendix (sampling settings of the evaluation: temperature 0.2,
                                  top-p 0.95): with temperature > 0 and 0 < top_p < 1, Sample draws
                                  from the most probable tokens up to the first at which the
                                  cumulative probability under softmax(logits / temperature) reaches
                                  top_p (equal logits at the cut stay together), renormalised;
                                  0 or 1 = off.  Needs vocab <= 65536 (else INVALID_ARG)          */
    int32_t latent_slots;      /* Appendix, "Larger Batch Sizes": number of slots for in-flight hidden
                                  states shared by all sequences of the session (the paper's "occupancy
                                  multiplier" times max_window).  0 or batch * max_window: every
                                  sequence owns max_window slots.  Fewer: slots are handed out from a
                                  pool as positions enter a wavefront and returned when they are
                                  committed; a sequence that finds the pool empty does not append a
                                  position that step (it stalls as at a full wavefront) and goes on
                                  when a slot is returned.  Slots go to sequences in index order.
                                  Needs batch <= 1024 (CAPACITY)                                   */
} rd_session_config;

typedef struct {
    uint64_t df_steps, ar_steps;           /* calls that enqueued work                       */
    uint64_t rows_prelude, rows_core, rows_coda; /* row-passes through P, R, C during decode
                                              (cost remark of Section 3.5)                   */
    uint64_t tokens_committed;             /* over all sequences, decode only                */
    uint64_t kernel_launches;              /* kernels of this library launched so far        */
    uint64_t tc_gemm_launches;             /* of those, tcgen05 GEMM launches                */
    /* Algorithmic work of the decode steps enqueued so far (what the method must move and compute,
     * cost remark of Section 3.5; not a measurement):                                         */
    uint64_t weight_bytes;                 /* every weight matrix once per pass: prelude, coda and
                                              head once per step, core and adapter once per inner
                                              iteration                                        */
    uint64_t kv_bytes;                     /* K and V: a sequence's cache rows 0..newest in-flight
                                              position read once per layer and pass for its whole
                                              window, plus the in-flight rows written          */
    uint64_t flops;                        /* 2 per weight element and row, plus 4 * hidden per
                                              (row, attended key, layer)                       */
    uint64_t commit_hist[16];              /* (step, live sequence) pairs by tokens committed in
                                              that step: [k] for k < 15, [15] for 15 or more   */
} rd_stats_t;

/* rd_load -- upload (or reference-free copy) of the weights of P, R, C (Section 3.1).
 *   cfg           host pointer.
 *   tensors       host array of pointers (each host or device memory), in this order:
 *                 emb [V,h]; for block in prelude, core, coda, for each layer: g1 [h], wq [h,h],
 *                 wk [h,h], wv [h,h], wo [h,h], g2 [h], wg [I,h], wu [I,h], wd [h,I];
 *                 adapter [h,2h] (columns 0..h-1 multiply e, h..2h-1 multiply s); g_core [h];
 *                 g_final [h]; head [V,h] only when tie_embeddings == 0.
 *                 Gains (g*) are float32.  Matrices are float32 when elem_bytes == 4 and bfloat16
 *                 bit patterns when elem_bytes == 2 (only valid with dtype RD_BF16); float32
 *                 input with dtype RD_BF16 is rounded to nearest-even once.
 *   n_tensors     length of `tensors` (checked against the shape).
 *   out           receives the model.  Errors: INVALID_ARG, OOM, CUDA. */
int rd_load(const rd_config* cfg, const void* const* tensors, int32_t n_tensors, int32_t elem_bytes,
            rd_model** out);
void rd_free(rd_model* m);

/* rd_session_create -- allocate KV caches (three blocks, [layer][sequence][head][position][head_dim]),
 * latent slots and token arrays for `batch` sequences.
 *   cuda_stream   a cudaStream_t (as void*) on which every step is enqueued; NULL = legacy
 *                 default stream.  The model must outlive the session.
 * The model's device must be the current device (STATE otherwise); the first session on a device
 * also sets that device's kernel attributes.  max_window may be at most 128 for RD_BF16 models whose
 * head_dim is 64, 96 or 128 to stay on the tensor-core attention kernel (wider windows, other head
 * sizes and RD_F32 run the one-row-per-block kernel).  batch * max_window <= 4096 (CAPACITY). */
int rd_session_create(const rd_model* m, const rd_session_config* sc, void* cuda_stream,
                      rd_session** out);
void rd_session_destroy(rd_session* s);

/* rd_prefill -- Section 3.3: positions 0..n_prompt-2 of sequence `seq` run P, `r` simultaneous
 * passes of R (pass i of position p attends pass-i K/V of positions <= p) and the coda layers;
 * position n_prompt-1 becomes the first in-flight position with a fresh state (the initialisation
 * steps of Algorithm 1).  prompt: host pointer to n_prompt token ids in [0, vocab); it is copied
 * before the call returns.  The call only ENQUEUES the work on the session's stream (upload of the
 * prompt, the passes, the sequence's new state) and returns; it allocates nothing.  Re-prefilling a
 * sequence restarts it; the other sequences of the session keep their wavefronts and go on with the
 * next step.  Errors: INVALID_ARG, CAPACITY (n_prompt + max_new_tokens > max_context), CUDA. */
int rd_prefill(rd_session* s, int32_t seq, const int32_t* prompt, int32_t n_prompt, int32_t r);

/* rd_prefill_sliced -- admission of a sequence into a running batch (Appendix, "Larger Batch Sizes":
 * new requests join between the steps of the sequences already decoding).  The result is that of
 * rd_prefill, bit for bit (same kernels on the same chunks in the same order), but the work is cut
 * into units -- one pass of P, R or the coda layers over one chunk of prompt rows (a chunk holds
 * max(512, decode rows of the session) rows, rounded up to a multiple of 16) -- and the steps that
 * follow work it off: each rd_df_step / rd_ar_step first enqueues `units_per_step` units
 * (rd_set_prefill_units; default 1) of the oldest pending job, so the running sequences are held
 * up by one unit per step instead of a whole prefill.  Until its last unit has
 * been enqueued, sequence `seq` is stopped: it has no in-flight rows, a step does nothing for it,
 * rd_committed / rd_poll_end report it as not done and leave it out of the seq = -1 totals (ask
 * rd_prefill_pending whether admissions are still under way).  The step whose units finish the job
 * is the first one the sequence takes part in.
 * The prompt is copied before the call returns; nothing is allocated.  Jobs are worked off in the
 * order of their registration.  A step called while no sequence is running only works on the jobs.
 * Errors: those of rd_prefill; STATE if `seq` already has a pending job.  While a job is pending
 * rd_prefill returns STATE (one prefill workspace per session).
 * rd_prefill_advance enqueues up to `units` units right away (no decode step), rd_prefill_pending
 * returns the number of jobs not yet finished (>= 0, or INVALID_ARG), rd_set_prefill_units sets the
 * units a step works off (0: steps leave the jobs to rd_prefill_advance). */
int rd_prefill_sliced(rd_session* s, int32_t seq, const int32_t* prompt, int32_t n_prompt, int32_t r);
int rd_prefill_advance(rd_session* s, int32_t units);
int rd_prefill_pending(const rd_session* s);
int rd_set_prefill_units(rd_session* s, int32_t units_per_step);

/* rd_ar_step -- one token on every live sequence by the sequential recurrence (Section 3.1):
 * e = P(newest token), s_0, r applications of R, p = C(s_r), sample, commit.
 * Errors: STATE (a sequence is not prefetched, or a wavefront wider than one is open). */
int rd_ar_step(rd_session* s, int32_t r);

/* rd_df_step -- one step of the diffusion-forcing sampler on every live sequence: e = P(y_current)
 * on the in-flight rows, `inner_iters` applications of R, drafts from C for every row, freeze and
 * commit the longest finished prefix, append one fresh position while fewer than `window` rows
 * are in flight.  exit_threshold <= 0: fixed exit (Algorithm 1; a row is finished after `window`
 * steps).  exit_threshold > 0: adaptive exit (Algorithm 2; finished when delta_i of Eq. 3 is below
 * the threshold, or after max_iters_per_pos core iterations).  With eta = beta = 0,
 * rd_df_step(1, r, 0) computes exactly what rd_ar_step(r) computes (rd_ar_step never applies the
 * stabilisers).  Errors: STATE, CAPACITY (window > max_window), INVALID_ARG. */
int rd_df_step(rd_session* s, int32_t window, int32_t inner_iters, float exit_threshold);

/* rd_sync -- wait for every enqueued step; returns TIMEOUT/CUDA if a kernel reported a fault. */
int rd_sync(rd_session* s);

/* rd_committed -- |y_frozen| of sequence `seq` (prompt + committed tokens); *done is set when the
 * sequence has produced max_new_tokens.  Either out pointer may be NULL. */
int rd_committed(rd_session* s, int32_t seq, int32_t* n_tokens, int32_t* done);

/* rd_poll_begin / rd_poll_end -- the same read without stalling the stream of steps.  rd_poll_begin
 * enqueues, behind the steps enqueued so far, a device-to-host copy of the session's polled state
 * (status word, |y_frozen| and done flag of every sequence) into one of two pinned buffers and returns
 * its ticket (0 or 1) at once.  rd_poll_end waits for that copy only and reports sequence `seq`
 * (seq = -1: *n_tokens = sum over the prefilled sequences, *done = all of them done).  A caller that
 * enqueues step t+1 between the two calls for step t keeps the device busy while it reads; steps on
 * finished sequences are no-ops, so running one step ahead is harmless.  At most two tickets are out
 * at a time (STATE otherwise).  rd_poll_end returns TIMEOUT when the status word was set. */
int rd_poll_begin(rd_session* s, int32_t* ticket);
int rd_poll_end(rd_session* s, int32_t ticket, int32_t seq, int32_t* n_tokens, int32_t* done);

/* rd_get_tokens -- copy up to `cap` tokens of y_frozen (prompt included) to host memory `dst`. */
int rd_get_tokens(rd_session* s, int32_t seq, int32_t* dst, int32_t cap, int32_t* n_written);

/* Inspection of the most recent step (rows are the positions that step processed, oldest first).
 * rd_last_step_rows gives their first position and count; rd_debug_read copies to host `dst`:
 *   RD_DBG_LATENTS float32 [n, hidden]   z after the step's last core iteration
 *   RD_DBG_DELTA   float32 [n]           delta_i of Eq. 3 against the state at the step's start
 *   RD_DBG_DRAFTS  int32   [n]           sampled tokens (row at position p drafts token p+1)
 *   RD_DBG_LOGITS  float32 [n, vocab]    needs keep_logits
 *   RD_DBG_EMBED   float32 [n, hidden]   e = P(y_current) of the step
 * `bytes` must be at least the size above, else INVALID_ARG. */
enum { RD_DBG_LATENTS = 0, RD_DBG_DELTA = 1, RD_DBG_DRAFTS = 2, RD_DBG_LOGITS = 3, RD_DBG_EMBED = 4 };
int rd_last_step_rows(rd_session* s, int32_t seq, int32_t* first_pos, int32_t* n_rows);
int rd_debug_read(rd_session* s, int32_t what, int32_t seq, void* dst, size_t bytes);

/* rd_debug_force_tokens -- overwrite y_current[first_pos .. first_pos+n) (drafts or the newest
 * committed tokens) from host memory; lets a lock-step comparison follow the other side through
 * a near-tie.  Positions inside the prompt are refused (INVALID_ARG). */
int rd_debug_force_tokens(rd_session* s, int32_t seq, int32_t first_pos, const int32_t* tokens,
                          int32_t n);

/* rd_debug_read_kv -- copy K (which=0) or V (which=1) of block (0 prelude, 1 core, 2 coda), layer,
 * sequence, positions [pos0, pos0+n) to host `dst` as float32 [n, hidden]. */
int rd_debug_read_kv(rd_session* s, int32_t block, int32_t layer, int32_t which, int32_t seq,
                     int32_t pos0, int32_t n, float* dst);

/* rd_debug_read_kv_noalloc -- rd_debug_read_kv for callers that must not allocate.  (The paper has
 * no counterpart: this is a property of the library, not of the method.)
 *
 * Who needs it: a serving process that sized its KV caches to take all the device memory that was
 * left, so a cudaMalloc of even a few megabytes fails; and a process that reads cache rows out while
 * other sessions keep stepping on other streams, where cudaMalloc / cudaFree would stall the whole
 * device for a moment.  rd_debug_read_kv takes a temporary float32 buffer from cudaMalloc on every
 * call; this call stages through a fixed array that is part of the library image instead and calls
 * no allocating routine.
 *
 * Arguments, layout of `dst` (host memory, float32 [n, hidden]) and results are those of
 * rd_debug_read_kv: the values are bit-identical.  Differences:
 *   - n * hidden may be at most 1,048,576 values (the staging array: 4 MiB, held by every device
 *     that loads the library until the process exits).  More is refused with RD_E_CAPACITY and a
 *     message in rd_last_cuda_error; nothing is read.
 *   - The session's device must be the current device (RD_E_STATE otherwise).
 *   - The first call on a device looks up the staging array's address on that device
 *     (cudaGetSymbolAddress) and remembers it; make that first call before any stream capture.
 *   - All calls on one device share the one staging array.  A call overwrites every value it later
 *     copies out, so the previous call's contents never show; but two calls that overlap in time on
 *     the same device (two host threads, two sessions) race on it: serialise them. */
int rd_debug_read_kv_noalloc(rd_session* s, int32_t block, int32_t layer, int32_t which, int32_t seq,
                             int32_t pos0, int32_t n, float* dst);

/* rd_debug_expire_next_wait -- test aid for the RD_E_TIMEOUT path.  Every wait of a GEMM kernel on a
 * pipeline barrier is bounded; when one runs out the kernel raises the session's status word, lets
 * the copies it issued land, frees its tensor memory and returns, and rd_sync reports RD_E_TIMEOUT
 * from then on (the session can still be destroyed, and other sessions are unaffected).  This call
 * makes that happen once: in the next tensor-core GEMM launch on single CTAs, one CTA never requests
 * the first operand tile of its share, so the barrier that tile would complete stays incomplete, and
 * the launch's waits give up after a few thousand polls instead of millions.  Nothing faults and no
 * wait is unbounded; the step's results are meaningless.  STATE when the session has no tensor-core
 * GEMM path. */
int rd_debug_expire_next_wait(rd_session* s);

/* rd_stats -- counters since session creation (host pointer out). */
int rd_stats(rd_session* s, rd_stats_t* out);

/* rd_profile_enable / rd_profile_read -- measurement aid.  While enabled, every GEMM launch, every
 * attention launch and every other kernel launch is bracketed by a pair of CUDA events recorded on
 * the session's stream (which also keeps consecutive kernels from overlapping);
 * rd_profile_read synchronises, sums the elapsed times of the pairs recorded since the last read
 * and resets the list.  Bytes are the algorithmic ones: weight bytes of each GEMM (n_out * K *
 * element size), and for attention the K and V rows each (sequence, layer) must read once.
 * At most 32768 pairs are kept between reads; later launches are then not bracketed. */
typedef struct {
    uint64_t gemm_launches;  double gemm_ms;  uint64_t gemm_weight_bytes;
    uint64_t attn_launches;  double attn_ms;  uint64_t attn_kv_bytes;
    uint64_t other_launches; double other_ms;
} rd_profile_t;
int rd_profile_enable(rd_session* s, int32_t on);
int rd_profile_read(rd_session* s, rd_profile_t* out);

/* rd_debug_gemm_sequence -- measurement aid: enqueues, `reps` times, the GEMM launches of one decode
 * step with one inner iteration (every layer's QKV, out, gate/up and down projection, the adapter, the
 * head; same shapes, operands, row tile and launch mode as in a step) with nothing between them, on
 * `n_rows` rows of the session's activation buffers as they stand (results unused; the session's
 * sequences are not touched, but a step enqueued later recomputes its activations anyway).  Timed
 * with events on the session's stream it gives the GEMM's launch duration inside a chain of launches,
 * without the gap that an event pair around a single launch adds.  *weight_bytes = algorithmic weight
 * bytes of the enqueued launches, *launches = their number.  RD_BF16 tensor-core path only (STATE). */
int rd_debug_gemm_sequence(rd_session* s, int32_t n_rows, int32_t reps, uint64_t* weight_bytes, int32_t* launches);

/* rd_set_gemm_path -- 0: SIMT kernels everywhere; 1 (default for RD_BF16): tcgen05 tensor-core
 * GEMMs where the shape allows, tiles of 128 and 256 rows on CTA pairs (one MMA of 256 features over
 * two SMs); 2: as 1 with those tiles on single CTAs.  For measurement and parity tests. */
int rd_set_gemm_path(rd_session* s, int32_t path);

/* rd_set_launch_chaining -- 1 (default): the kernels of a step are launched as a programmatic-
 * dependent-launch chain (each may start, and prefetch weights, while its predecessor finishes);
 * 0: ordinary stream-ordered launches.  Results are identical; for measurement and tests. */
int rd_set_launch_chaining(rd_session* s, int32_t on);

/* rd_set_attention_path -- 3 (default for RD_BF16 with head_dim 64, 96 or 128): as 2, and prefill
 * (groups of 128 consecutive prompt rows) with both products on tcgen05, S and O in tensor memory;
 * 2: windowed tensor-core attention (mma.sync) with K and V brought in by TMA through a ring of
 * barrier-guarded stages (groups of at most
 * 8 rows, e.g. the sequential decoder's one row per sequence, take the cp.async kernel); 1: the same
 * arithmetic with K and V brought in by cp.async, double buffered; 0: one block per (row, head).
 * For measurement (A/B) and tests.  STATE when the model cannot take the requested path. */
int rd_set_attention_path(rd_session* s, int32_t path);

/* rd_set_fused_swiglu -- 1 (default): on the tensor-core path the gate/up projection runs on whole
 * tiles and its epilogue writes silu(gate) * up directly (no partial sums, no separate kernel);
 * 0: the projection leaves partial sums and a separate kernel applies the SwiGLU.  Same arithmetic up
 * to the order of the float32 sums; for measurement (A/B) and tests. */
int rd_set_fused_swiglu(rd_session* s, int32_t on);

const char* rd_strerror(int code);
/* Text of the last CUDA error this library saw on the calling thread's most recent failing call
 * (static storage, never NULL). */
const char* rd_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* RD_H_ */
