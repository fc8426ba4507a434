/*
 * spec_verify -- verify-and-resample pass of speculative sampling on NVIDIA B200
 * (sm_100a).  C ABI: plain pointers and sizes, no C++ or framework types.
 *
 * The operation is the one the paper's section "Speculative Sampling Results"
 * describes for each speculation round: the draft model has proposed K tokens;
 * the target model has scored K+1 positions; the two models' probabilities of
 * the proposed tokens are compared, a rejection criterion decides how many
 * proposed tokens are kept, the first rejected token is resampled from a
 * combination of the two distributions, and if nothing was rejected one more
 * token is sampled from the target's distribution.  The per-sequence lookahead
 * K_b may differ between sequences (the paper's input-dependent speculation,
 * section "Dynamic Execution").  The paper gives no formulas; this library
 * uses the rule of the speculative-sampling papers it cites:
 *
 *   p_i = softmax(target_logits[b,i,:] / T_b),  q_i = softmax(draft_logits[b,i,:] / T_b)
 *   draft token x_i is accepted iff  u_i < p_i(x_i) / q_i(x_i)   (evaluated as u_i*q < p)
 *   n_b = first rejected position (K_b if none)
 *   n_b < K_b : emit  j ~ max(0, p_n - q_n) / sum  by inverse CDF with u'_b
 *   n_b = K_b : emit  j ~ p_K                      by inverse CDF with u'_b
 *   inverse CDF: smallest j whose inclusive cumulative mass is > u' * total
 *
 * Packed ragged layout.  With off_d[b] = sum_{c<b} max(K_c,0) and
 * off_t[b] = off_d[b] + b:
 *   target_logits  [n_draft_total + B][ld_target]  row off_t[b]+i, i in [0,K_b]
 *   draft_logits   [n_draft_total    ][ld_draft ]  row off_d[b]+i, i in [0,K_b)
 *   draft_tokens   [n_draft_total]                 entry off_d[b]+i
 *   uniforms       [n_draft_total + B]             entry off_t[b]+i (i<K_b) is u_i,
 *                                                  entry off_t[b]+K_b is u'_b
 *   emitted_tokens [n_draft_total + B]             entries off_t[b]..off_t[b]+K_b:
 *                                                  n_b accepted draft tokens, the
 *                                                  sampled token, then -1
 * Only the first V elements of a logits row are read; ld_* >= V is the row
 * pitch in elements.
 *
 * Every function returns a specv_status (0 = success) unless stated otherwise.
 * Nothing here allocates or frees device memory, synchronises the device, or
 * reads device memory from the host, except where a function says so.
 */
#ifndef SPEC_VERIFY_H
#define SPEC_VERIFY_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum { SPECV_F32 = 0, SPECV_BF16 = 1, SPECV_F16 = 2 } specv_dtype;

typedef enum {
    SPECV_OK = 0,
    SPECV_ERR_NULL = 1,       /* a required pointer is NULL */
    SPECV_ERR_SHAPE = 2,      /* B, V, ld, k_uniform or n_draft_total out of range */
    SPECV_ERR_DTYPE = 3,      /* dtype is not a specv_dtype */
    SPECV_ERR_ALIGN = 4,      /* workspace / int / float pointer not aligned to its type */
    SPECV_ERR_WORKSPACE = 5,  /* workspace or arena smaller than required */
    SPECV_ERR_CUDA = 6,       /* a CUDA call failed; see spec_verify_last_cuda_error */
    SPECV_ERR_ARCH = 7,       /* the current device is not compute capability 10.x */
    SPECV_ERR_TOO_LARGE = 8,  /* spec_verify_noalloc only: batch exceeds the built-in scratch */
    SPECV_ERR_FLAGS = 9       /* unknown flag bits, both kernel-set bits, or a flag the call does not take */
} specv_status;

/* Per-call options (`flags` arguments).  The library keeps no mode between calls: two host threads
 * may run passes with different options at the same time (on different workspaces). */
enum {
    SPECV_FLAG_STREAMING = 1,   /* use the streaming kernels (any shape) */
    SPECV_FLAG_RING = 2,        /* use the ring kernels (bulk async copies into a shared-memory ring, the
                                   batch cut into equal byte ranges per SM) whenever the shape allows them:
                                   rows on 16-byte boundaries, V*elt a multiple of 16, V at most 2^19
                                   elements for bf16 / fp16 and 2^18 for fp32, at most 4095 sequences;
                                   else streaming.  Neither bit: automatic, the ring kernels from 64
                                   target rows up.  Results of the two sets agree except for draws within
                                   rounding of a decision boundary. */
    SPECV_FLAG_EARLY_EXIT = 4,  /* spec_verify_ex only; see there */
    SPECV_FLAG_CLUSTER = 8      /* the one-launch form for small batches: a thread-block cluster of eight
                                   CTAs per sequence keeps all of the sequence's logits rows in shared
                                   memory (every logit fetched once, no workspace traffic).  Taken when
                                   the batch has at most 18 sequences, rows on 16-byte boundaries with
                                   V*elt a multiple of 16, a lookahead of at most 32 (if k_per_row is
                                   given the host cannot see it and n_draft_total must be at most 32),
                                   and (2K+1) rows of ceil(V*elt/512/8)*512 bytes fit in 200 KB; else
                                   the automatic choice.  The automatic choice (no kernel-set bit)
                                   takes this form whenever those conditions hold. */
};

/* Bits of row_status[b] (data errors found on the device; the call itself succeeds).
 * With any of the first three set the sequence yields accepted_len 0 and -1 tokens. */
enum {
    SPECV_ROW_BAD_K = 1,            /* K_b < 0, or the sequence's rows overrun n_draft_total */
    SPECV_ROW_BAD_TEMPERATURE = 2,  /* T_b not finite or <= 0 */
    SPECV_ROW_BAD_TOKEN = 4,        /* a draft token outside [0, V) */
    SPECV_ROW_ZERO_RESIDUAL = 8,    /* sum max(0,p-q) rounded to 0 at the rejection: the token
                                       was sampled from p_n instead (output still valid) */
    SPECV_ROW_INTERNAL = 16,        /* a bounded wait inside a ring kernel expired (should never
                                       happen); the sequence yields accepted_len 0 and -1 tokens;
                                       bits 8 and up then name the wait */
    SPECV_ROW_BAD_PARENT = 32       /* spec_verify_tree: a parent index outside [-1, own index);
                                       the sequence yields accepted_len 0 and -1 tokens */
};

/* Text for a specv_status; never NULL; static storage. */
const char* spec_verify_strerror(int status);

/* cudaError_t value of the most recent failed CUDA call made by this library on the
 * calling thread (0 if none). */
int spec_verify_last_cuda_error(void);

/* Number of kernels this library has launched since it was loaded (all threads). */
uint64_t spec_verify_launch_count(void);

/*
 * Bytes of device scratch that spec_verify needs for a batch of B sequences with
 * n_draft_total drafted positions over a vocabulary of V.  Depends on nothing else.
 * Returns 0 for arguments that spec_verify would reject.
 */
size_t spec_verify_workspace_bytes(int32_t B, int64_t n_draft_total, int64_t V);

/*
 * One verify-and-resample pass over a batch (steps: softmax statistics of every
 * logits row, acceptance ratios of all draft positions in parallel, first rejection,
 * residual or bonus sample, emit).  All data pointers are DEVICE pointers on the
 * current device; the caller owns every buffer, including the workspace, and must keep
 * them alive and unmodified until the work enqueued on cuda_stream has finished.
 *
 *   target_logits, draft_logits  packed rows (see top), element type `dtype`; any
 *                                alignment and pitch are accepted, 16-byte aligned
 *                                rows take the vectorised path
 *   V, ld_target, ld_draft       in elements; 1 <= V <= ld_*; V < 2^31
 *   draft_tokens                 int32 [n_draft_total]; may be NULL iff n_draft_total == 0
 *   k_per_row                    int32 [B], or NULL: every sequence has k_uniform drafts
 *   B, k_uniform, n_draft_total  host scalars; B >= 1; with k_per_row == NULL,
 *                                n_draft_total must equal B * k_uniform
 *   temperature                  float [B] if temperature_per_row, else float [1]
 *   uniforms                     float [n_draft_total + B], values in [0,1)
 *   accepted_len                 out, int32 [B]
 *   emitted_tokens               out, int32 [n_draft_total + B]; every entry is written
 *   row_status                   out, int32 [B], may be NULL
 *   diag_p_tok, diag_q_tok       out, float [n_draft_total], may be NULL: p_i(x_i), q_i(x_i)
 *                                for every draft position (also those after the rejection)
 *   workspace, workspace_bytes   device scratch, 256-byte aligned,
 *                                >= spec_verify_workspace_bytes(B, n_draft_total, V);
 *                                contents need not be initialised and are clobbered
 *   cuda_stream                  cudaStream_t (NULL = the default stream)
 *
 * The call validates the host-visible arguments, enqueues its kernels on cuda_stream and
 * returns without waiting; outputs are valid once the stream reaches that point.  The first call
 * on a device for a given dtype also sets kernel attributes; from the second on, a call only
 * enqueues kernels and may be captured in a CUDA graph (stream capture) and replayed.  Two
 * calls may overlap on the device only if they use different workspaces.  Argument errors
 * are reported before anything is launched; a failed launch returns SPECV_ERR_CUDA.  Bad
 * DATA (see SPECV_ROW_*) never faults: it is reported per sequence in row_status.
 */
int spec_verify(const void* target_logits, const void* draft_logits, int dtype,
                int64_t V, int64_t ld_target, int64_t ld_draft,
                const int32_t* draft_tokens, const int32_t* k_per_row,
                int32_t B, int32_t k_uniform, int64_t n_draft_total,
                const float* temperature, int temperature_per_row,
                const float* uniforms,
                int32_t* accepted_len, int32_t* emitted_tokens, int32_t* row_status,
                float* diag_p_tok, float* diag_q_tok,
                void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * spec_verify with per-call options and, optionally, the lookahead of the next speculation round
 * written by the same kernels.  spec_verify(...) is spec_verify_ex(..., 0, 0, 0, NULL).
 *
 *   flags   SPECV_FLAG_STREAMING, SPECV_FLAG_RING or SPECV_FLAG_CLUSTER (kernel set; none: automatic), and
 *           SPECV_FLAG_EARLY_EXIT: the paper's theme is to do only the work the input needs; in this
 *           pass nothing after a sequence's first rejected draft token can be emitted, so the logits
 *           rows of later positions need not be read.  With this flag the ring kernels process the
 *           positions of all sequences in order (position 0 of every sequence first) and skip every
 *           row pair that lies after a position already rejected with a clear margin.  accepted_len,
 *           emitted_tokens and row_status are exactly those of the normal mode; diag_p_tok /
 *           diag_q_tok are NaN at skipped positions.  Ignored whenever the streaming kernels run.
 *   next_k  device out, int32 [B], may be NULL: the lookahead for the next round (the paper's
 *           input-dependent speculation, sections "Dynamic Execution" and "Speculative Sampling
 *           Results"; the paper gives no rule, this is a stated heuristic): K_b + 2 if every drafted
 *           token of sequence b was accepted, else K_b - 1, clamped to [k_min, k_max]; for a sequence
 *           with a data error accepted_len counts as 0 and a negative K_b as 0.  Written by the warp
 *           that emits the sequence's tokens; it never influences which tokens are emitted.
 *   k_min, k_max   used only with next_k: 0 <= k_min <= k_max, else SPECV_ERR_SHAPE.
 * Unknown flag bits or both kernel-set bits: SPECV_ERR_FLAGS.  Everything else as for spec_verify.
 */
int spec_verify_ex(const void* target_logits, const void* draft_logits, int dtype,
                   int64_t V, int64_t ld_target, int64_t ld_draft,
                   const int32_t* draft_tokens, const int32_t* k_per_row,
                   int32_t B, int32_t k_uniform, int64_t n_draft_total,
                   const float* temperature, int temperature_per_row,
                   const float* uniforms,
                   int32_t* accepted_len, int32_t* emitted_tokens, int32_t* row_status,
                   float* diag_p_tok, float* diag_q_tok,
                   void* workspace, size_t workspace_bytes, void* cuda_stream,
                   uint32_t flags, int32_t k_min, int32_t k_max, int32_t* next_k);

/* Kernel set the calling thread's most recent pass (any entry point below or above) used:
 * 1 streaming, 2 ring, 3 the one-launch cluster form, 0 if it has made none.  Not a status code. */
int spec_verify_last_path(void);

/*
 * Optional per-kernel timing for profiling runs.  `events` points to 4 cudaEvent_t
 * handles created by the caller (timing enabled); while set, every spec_verify call made
 * by the calling thread records events[0] before its first kernel, events[1] before the
 * row-statistics kernel, events[2] before the resolve kernel and events[3] after it, on
 * the call's stream (the ring kernel set has no kernel before the statistics kernel: events[0]
 * and events[1] are then recorded back to back).  Recording between the kernels also switches
 * off their overlap.  NULL switches it off (the default).  The handles are only stored;
 * the caller keeps ownership.  Always returns SPECV_OK.
 */
int spec_verify_set_trace_events(void* const* events);

/*
 * Lookahead for the next speculation round (the paper's input-dependent speculation, sections
 * "Dynamic Execution" and "Speculative Sampling Results"; the paper gives no rule, this is a
 * stated heuristic): next_k[b] = K_b + 2 if every drafted token of sequence b was accepted
 * (accepted_len[b] >= K_b), else K_b - 1, clamped to [k_min, k_max].  It never influences
 * which tokens are emitted.  k_per_row (or NULL with k_uniform), accepted_len and next_k are
 * DEVICE int32 arrays of B entries; one small kernel is enqueued on cuda_stream (spec_verify_ex can
 * write the same values from inside the pass, without this extra launch).  Returns
 * SPECV_ERR_NULL / SPECV_ERR_SHAPE (B < 1, k_min < 0, k_max < k_min) / SPECV_ERR_CUDA.
 */
int spec_verify_next_lookahead(const int32_t* k_per_row, int32_t k_uniform, const int32_t* accepted_len,
                               int32_t B, int32_t k_min, int32_t k_max, int32_t* next_k, void* cuda_stream);

/*
 * Tree-structured verification.  The draft proposes, per sequence, a TREE of candidate tokens
 * (several candidates for the same position; the paper's section "Speculative Sampling Results"
 * lists tree drafting among the methods it builds on) and the target scores every node in one
 * pass.  The verifier walks from the root; the rule is the recursive rejection sampling of those
 * methods, which keeps the emitted tokens distributed exactly as the target's when the children
 * of a context are independent draws from the draft distribution of that context:
 *
 *   at context c (0 = the root, j+1 = the context after node j) let r = p_c;
 *   for each child j of c in increasing node index, with token x_j and uniform u_j:
 *       accept j  iff  u_j < r(x_j) / q_c(x_j)       (evaluated as u_j * q_c(x_j) < r(x_j));
 *       accepted: emit x_j and continue at context j+1;
 *       rejected: r <- max(0, r - q_c) / sum_v max(0, r(v) - q_c(v)), try the next child;
 *   when no child is accepted (or c has none) emit one token drawn from r by inverse CDF with
 *   the sequence's last uniform, and stop.
 * p_c = softmax(target row of c / T_b), q_c = softmax(draft row of c / T_b).  A chain (node j the
 * only child of node j-1) gives exactly spec_verify.  A residual that rounds to zero leaves r as
 * it was and sets SPECV_ROW_ZERO_RESIDUAL.
 *
 * Layout, with N_b nodes in sequence b, off_d[b] = sum_{c<b} max(N_c,0), off_t[b] = off_d[b] + b:
 *   target_logits  [n_node_total + B][ld_target]  row off_t[b]+c: context c, c in [0, N_b]
 *   draft_logits   [n_node_total    ][ld_draft ]  row off_d[b]+c: the distribution the children of
 *                                                 context c were drawn from; rows of contexts
 *                                                 without children are never read
 *   node_tokens, node_parent [n_node_total]       entry off_d[b]+j; parent -1 = the root, else the
 *                                                 index (within the sequence) of a node < j
 *   n_per_seq [B] or NULL with n_uniform          N_b
 *   uniforms       [n_node_total + B]             entry off_t[b]+j: u_j; entry off_t[b]+N_b: the last uniform
 *   emitted_tokens [n_node_total + B]             entries off_t[b]..: tokens of the accepted path, the
 *                                                 drawn token, then -1
 *   accepted_nodes [n_node_total + B], may be NULL  entries off_t[b]..: node index of each accepted
 *                                                 token, -1 elsewhere
 *   accepted_len [B]                              nodes on the accepted path
 *   diag_p_tok, diag_q_tok [n_node_total], may be NULL  p_c(x_j), q_c(x_j) of EVERY node j, c the
 *                                                 context of its parent
 *   workspace                                     >= spec_verify_tree_workspace_bytes(B, n_node_total, V)
 *   flags                                         SPECV_FLAG_STREAMING / SPECV_FLAG_RING or 0 (kernel set of
 *                                                 the row statistics); SPECV_FLAG_EARLY_EXIT is refused
 * Everything else (pointers are DEVICE pointers, dtype, temperature, row_status, asynchrony, error
 * reporting) as for spec_verify.  Each rejected child costs one more pass
 * over its context's two rows; the row statistics are computed once for every row that is needed.
 */
size_t spec_verify_tree_workspace_bytes(int32_t B, int64_t n_node_total, int64_t V);
int spec_verify_tree(const void* target_logits, const void* draft_logits, int dtype,
                     int64_t V, int64_t ld_target, int64_t ld_draft,
                     const int32_t* node_tokens, const int32_t* node_parent, const int32_t* n_per_seq,
                     int32_t B, int32_t n_uniform, int64_t n_node_total,
                     const float* temperature, int temperature_per_seq, const float* uniforms,
                     int32_t* accepted_len, int32_t* emitted_tokens, int32_t* accepted_nodes,
                     int32_t* row_status, float* diag_p_tok, float* diag_q_tok,
                     void* workspace, size_t workspace_bytes, void* cuda_stream, uint32_t flags);

/*
 * Greedy verification: the temperature -> 0 limit of the pass above (the paper's section
 * "Speculative Sampling Results" describes the sampled form only).  Both softmaxes become one-hot
 * at their row's largest logit, so draft logits, temperature and uniforms drop out:
 *
 *   draft token x_i is accepted iff  x_i == argmax_j target_logits[b,i,j]
 *   n_b = first mismatch (K_b if none); the token emitted after the accepted prefix is
 *   argmax_j target_logits[b,n_b,j]  (the residual is one-hot there; for n_b = K_b the bonus token)
 *
 * Among equal largest logits the smallest token id is the argmax; a NaN logit is never the
 * largest; a row with nothing above -inf gives token 0.  Results are exact (no rounding is
 * involved).  Only the target rows are read, each once.
 *
 * Layout, B / k_per_row / k_uniform / n_draft_total, accepted_len, emitted_tokens, row_status
 * (bits SPECV_ROW_BAD_K, SPECV_ROW_BAD_TOKEN, SPECV_ROW_INTERNAL), asynchrony and error
 * reporting as for spec_verify; all data pointers are DEVICE pointers.
 *   target_argmax              out, int32 [n_draft_total + B], may be NULL: argmax of every target
 *                              row, in target packing
 *   workspace, workspace_bytes device scratch, 256-byte aligned,
 *                              >= spec_verify_greedy_workspace_bytes(B, n_draft_total); need not
 *                              be initialised, clobbered
 *   flags                      SPECV_FLAG_STREAMING / SPECV_FLAG_RING or 0: the ring kernel (bulk async
 *                              copies) needs rows on 16-byte boundaries with V*elt a multiple of 16 and
 *                              is chosen automatically from 64 target rows up
 */
size_t spec_verify_greedy_workspace_bytes(int32_t B, int64_t n_draft_total);
int spec_verify_greedy(const void* target_logits, int dtype, int64_t V, int64_t ld_target,
                       const int32_t* draft_tokens, const int32_t* k_per_row,
                       int32_t B, int32_t k_uniform, int64_t n_draft_total,
                       int32_t* accepted_len, int32_t* emitted_tokens, int32_t* row_status,
                       int32_t* target_argmax,
                       void* workspace, size_t workspace_bytes, void* cuda_stream, uint32_t flags);

/*
 * The verify pass fed with HIDDEN STATES instead of logits: the step in front of it fused with its
 * first half.  The paper's section "Speculative Sampling Results" has the target model score the
 * drafted positions in one parallel pass (and the draft model before it); the output of those passes
 * -- logits = hidden x weight^T of each model's output layer -- is what the verify pass reads.
 * Here the two products run on the tensor cores (bf16 inputs, fp32 accumulation, results rounded to
 * bf16) and the row statistics of the verify pass -- (reference, sum) of 2^(logit * log2(e)/T - reference)
 * over the vocabulary, taken from the ROUNDED logits -- are computed in the products' epilogue, while
 * the accumulators are still on chip.  The logits are written once, to the caller's buffers (the
 * resolve step reads the one or two rows per sequence a token is drawn from, and the caller may want
 * them), and never read back for the statistics.  Results are those of spec_verify on the logits
 * this call writes (ring kernels).
 *
 *   target_hidden  bf16 [n_draft_total + B, ld_th]  hidden state of every target row (packing of target_logits)
 *   target_weight  bf16 [V, ld_tw]                  output-layer weight of the target model, row v = token v
 *   draft_hidden   bf16 [n_draft_total, ld_dh], draft_weight bf16 [V, ld_dw]   the same for the draft model
 *   H_target, H_draft                               hidden sizes (>= 1); ld_* >= H in elements
 *   target_logits  out, bf16 [n_draft_total + B, ld_target];  draft_logits out, bf16 [n_draft_total, ld_draft]
 * All four inputs: DEVICE pointers on 16-byte boundaries with pitches that are multiples of 16 bytes
 * (tensor-map loads); the logits buffers as the ring kernels want them (rows on 16-byte boundaries,
 * V * 2 a multiple of 16, V <= 2^19, B <= 4095) -- else SPECV_ERR_SHAPE.  Everything else
 * (draft_tokens .. diag_q_tok, asynchrony, error reporting) as for spec_verify;
 * workspace >= spec_verify_from_hidden_workspace_bytes(B, n_draft_total, V).
 * spec_verify_from_hidden_status reads back (after waiting for cuda_stream) the status word of the
 * product kernels of the last call on that workspace: 0, or the code of a bounded wait that expired.
 */
size_t spec_verify_from_hidden_workspace_bytes(int32_t B, int64_t n_draft_total, int64_t V);
int spec_verify_from_hidden(const void* target_hidden, int64_t ld_th, int64_t H_target,
                            const void* target_weight, int64_t ld_tw,
                            const void* draft_hidden, int64_t ld_dh, int64_t H_draft,
                            const void* draft_weight, int64_t ld_dw, int64_t V,
                            void* target_logits, int64_t ld_target, void* draft_logits, int64_t ld_draft,
                            const int32_t* draft_tokens, const int32_t* k_per_row,
                            int32_t B, int32_t k_uniform, int64_t n_draft_total,
                            const float* temperature, int temperature_per_row, const float* uniforms,
                            int32_t* accepted_len, int32_t* emitted_tokens, int32_t* row_status,
                            float* diag_p_tok, float* diag_q_tok,
                            void* workspace, size_t workspace_bytes, void* cuda_stream);
int spec_verify_from_hidden_status(const void* workspace, int32_t B, int64_t n_draft_total, int64_t V,
                                   void* cuda_stream);

/*
 * Self-test of the bounded waits (a diagnostic; the paper has no counterpart).  Every wait inside
 * the ring kernels -- on a shared-memory barrier that a bulk copy or another warp completes --
 * carries a limit of about a second; past it the wait gives up, records which wait it was, every
 * other wait of the thread block returns at once, and the kernel ends in bounds with
 * SPECV_ROW_INTERNAL in row_status.  This entry point runs that mechanism on purpose, harmlessly:
 * one small kernel whose first warp waits, with the given limit, on a barrier that nothing ever
 * completes.  out4 is a DEVICE array of four int64: [0] the error word (77: the first wait gave
 * up), [1] clock cycles the first wait lasted (just over the limit), [2] cycles of a second wait
 * on another barrier (a few hundred: it returns because the block has already failed), [3] 1 once
 * the kernel has reached its end.  limit_cycles in [1, 2e9]; else SPECV_ERR_SHAPE.
 */
int spec_verify_selftest_bounded_wait(int64_t limit_cycles, int64_t* out4, void* cuda_stream);

/*
 * Debug aid (the paper has no counterpart).  A library built with -DSPECV_DEBUG
 * (python -m paper_2411_00853_b200.build --debug -> libspecverify_debug.so) range-checks every row
 * index, split number, segment number and token id that the streaming kernels compute, before use;
 * a violation is recorded and the access skipped, nothing traps.  Returns the largest site code
 * recorded on the current device since the library was loaded (0: none; waits for the device),
 * -1 from a library built without the checks, -2 if the value could not be read.
 */
int spec_verify_debug_violation(void);

/*
 * Bytes of device memory ("arena") that spec_verify_host needs: device copies of all
 * inputs and outputs with dense pitch (ld = V) plus the workspace.  0 for arguments that
 * would be rejected.
 */
size_t spec_verify_host_arena_bytes(int dtype, int32_t B, int64_t n_draft_total, int64_t V);

/*
 * The same pass for callers whose data lives in HOST memory: copies the inputs to the
 * device arena, runs spec_verify, copies accepted_len, emitted_tokens (and row_status,
 * diag_* when given) back, and waits for cuda_stream before returning, so the outputs
 * are valid on return.  All data pointers are HOST pointers with the shapes above
 * (pinned memory makes the copies asynchronous to the host but is not required);
 * `arena` is a DEVICE pointer, 256-byte aligned, of at least
 * spec_verify_host_arena_bytes(...) bytes, owned by the caller and clobbered.
 * Logits rows are copied with their pitch removed.  `flags` as for spec_verify_ex (0: automatic
 * kernel set, normal mode).  Errors as for spec_verify_ex; a failed copy or synchronisation returns
 * SPECV_ERR_CUDA.
 */
int spec_verify_host(const void* target_logits, const void* draft_logits, int dtype,
                     int64_t V, int64_t ld_target, int64_t ld_draft,
                     const int32_t* draft_tokens, const int32_t* k_per_row,
                     int32_t B, int32_t k_uniform, int64_t n_draft_total,
                     const float* temperature, int temperature_per_row,
                     const float* uniforms,
                     int32_t* accepted_len, int32_t* emitted_tokens, int32_t* row_status,
                     float* diag_p_tok, float* diag_q_tok,
                     void* arena, size_t arena_bytes, void* cuda_stream, uint32_t flags);

/*
 * spec_verify for callers that must not allocate device memory.  (No counterpart in the
 * paper: this is a packaging variant of the call above, added for deployment.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- a serving process whose
 * memory pool already owns all of HBM, so a fresh allocation fails or fragments it; a plug-in
 * whose host application forbids allocation calls inside its callbacks; a latency-critical
 * decode loop that cannot afford the device-wide synchronisation an allocation may imply.
 * Such a caller has nowhere to get the `workspace` of spec_verify from.  Here the scratch is a
 * fixed array of SPECV_NOALLOC_SCRATCH_BYTES bytes compiled into the library's device image;
 * each GPU that loads the library carries it until the process exits.  The call itself makes
 * no allocation of any kind (no cudaMalloc/cudaFree, no allocating library routine).
 *
 * Arguments, layout, outputs, asynchrony and error reporting are exactly those of
 * spec_verify, without `workspace` / `workspace_bytes`.  The same kernels run as for spec_verify on
 * the same batch (same automatic choice of the kernel set), so the results are bit-identical to
 * spec_verify's.  Differences:
 *   - Size limit: spec_verify_workspace_bytes(B, n_draft_total, V) must not exceed
 *     SPECV_NOALLOC_SCRATCH_BYTES (4 MiB -- e.g. 64 sequences x 8 drafts over a vocabulary of
 *     128256 need 0.3 MiB, 256 x 4 over 152064 need 1.3 MiB; the size grows with B * V);
 *     larger batches are refused with SPECV_ERR_TOO_LARGE before anything is launched.
 *   - First call on each device looks up the array's device address (once per device, with
 *     that device current).  Make that first call outside any stream capture.
 *   - All calls on a device share the one array, and it keeps whatever the previous call left
 *     in it.  Nothing in it needs to be zero on entry (each call writes every word, the tickets
 *     and counters that must start at zero included, before reading it), but two calls whose kernels overlap on the GPU -- different streams, or
 *     different host threads -- would overwrite each other's scratch: serialise them (same
 *     stream, or an event between them).
 */
#define SPECV_NOALLOC_SCRATCH_BYTES (4u << 20)
int spec_verify_noalloc(const void* target_logits, const void* draft_logits, int dtype,
                        int64_t V, int64_t ld_target, int64_t ld_draft,
                        const int32_t* draft_tokens, const int32_t* k_per_row,
                        int32_t B, int32_t k_uniform, int64_t n_draft_total,
                        const float* temperature, int temperature_per_row,
                        const float* uniforms,
                        int32_t* accepted_len, int32_t* emitted_tokens, int32_t* row_status,
                        float* diag_p_tok, float* diag_q_tok, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* SPEC_VERIFY_H */
