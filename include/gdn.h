/*
 * libgdn -- gated delta-rule recurrence of Gated DeltaNet for NVIDIA B200 (sm_100a).
 *
 * For every sequence (or batch item) and value head h, with hq = h / (Hv / Hqk):
 *
 *     S_t = alpha_t S_{t-1} (I - beta_t k_t k_t^T) + beta_t v_t k_t^T ,   alpha_t = exp(g_t)
 *     o_t = S_t q_t
 *
 * i.e. decay the state, read old_v = S k, form delta = beta (v - old_v), add the
 * rank-one update delta k^T, and read the output from the updated state (the paper's
 * Section 3.2 equations, with the state stored transposed: [dv][dk], dk contiguous).
 *
 * Conventions shared by every entry point
 *   - Every data pointer is a DEVICE pointer unless stated otherwise.  The caller owns
 *     all buffers (destination passing: outputs are pre-allocated by the caller); the
 *     library allocates no device memory and keeps no reference after it returns.
 *   - Calls enqueue work on `stream` (a cudaStream_t passed as void*, NULL = default
 *     stream) and return without synchronising.
 *   - Return value: GDN_OK (0) or a positive gdn_status; on error nothing is enqueued.
 *     No exceptions, no aborts, no printing.
 *   - bf16 tensors are passed as `const void*` (2-byte elements); 16-byte alignment is
 *     required for every tensor pointer.
 *   - Only dk = dv = 128 is supported; Hv must be a multiple of Hqk (value heads
 *     h = j*G .. j*G+G-1 share q/k head j, G = Hv/Hqk).
 *   - gdn_decode / gdn_prefill take the log-decay g (alpha = exp(g)) and the write strength
 *     beta, both per value head, use q and k as given, and apply no scale: o = S q literally.
 *     The *_gated entry points compute g and beta from the raw gate inputs inside the kernels;
 *     the *_fused entry points additionally L2-normalise q and k and scale q (see there).
 */
#ifndef GDN_H_
#define GDN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum gdn_status {
    GDN_OK = 0,
    GDN_ERR_NULL = 1,        /* a required pointer is NULL                                   */
    GDN_ERR_SHAPE = 2,       /* negative size, Hv % Hqk != 0, max_seqlen inconsistent        */
    GDN_ERR_UNSUPPORTED = 3, /* dk != 128 or dv != 128, or the device is not sm_100          */
    GDN_ERR_WORKSPACE = 4,   /* workspace NULL, too small or not 1024-byte aligned           */
    GDN_ERR_ALIGN = 5,       /* a tensor pointer is not 16-byte aligned                      */
    GDN_ERR_CUDA = 6         /* the CUDA runtime reported an error while enqueueing          */
} gdn_status;

/* Human-readable name of a status code (static storage, never NULL). */
const char* gdn_status_string(int status);

/*
 * Single-token decode (Section 3.2: old_v, delta, S' and out, one token per batch item).
 * Reads each state row once and writes it once in the same pass; the output uses
 * out = q^T(alpha S) + delta (q^T k), so the updated state is never re-read.
 *
 *   q, k      bf16 [B, Hqk, dk]
 *   v         bf16 [B, Hv, dv]
 *   g, beta   fp32 [B, Hv]
 *   state_in  fp32 [B, Hv, dv, dk]
 *   state_out fp32 [B, Hv, dv, dk]   may be exactly state_in (in place); partial overlap is
 *                                    undefined
 *   out       bf16 [B, Hv, dv]       rounded to nearest even from fp32
 *
 * B = 0 returns GDN_OK without launching.
 */
int gdn_decode(const void* q, const void* k, const void* v, const float* g, const float* beta,
               const float* state_in, float* state_out, void* out,
               int B, int Hqk, int Hv, int dk, int dv, void* stream);

/*
 * gdn_decode with an explicit launch shape (rows per warp x warps per CTA), for tuning
 * the batch-regime table of Section 5.4 ("decode gap: dispatch and shape split").
 * variant in [0, gdn_decode_num_variants()); same arguments and result as gdn_decode.
 */
int gdn_decode_variant(const void* q, const void* k, const void* v, const float* g, const float* beta,
                       const float* state_in, float* state_out, void* out,
                       int B, int Hqk, int Hv, int dk, int dv, int variant, void* stream);
int gdn_decode_num_variants(void);

/*
 * Multi-token decode (the "multi-token decode" regime of Section 5.4's dispatch discussion):
 * T tokens per batch item, applied in order by the per-token recurrence of Section 3.2 to state
 * rows held in registers, so the state is still read once and written once per call.
 *
 *   q, k      bf16 [B, T, Hqk, dk]
 *   v, out    bf16 [B, T, Hv, dv]
 *   g, beta   fp32 [B, T, Hv]
 *   state_in / state_out  fp32 [B, Hv, dv, dk]   (may alias exactly)
 *
 * T = 0 copies state_in to state_out; T = 1 is gdn_decode.
 */
int gdn_decode_multi(const void* q, const void* k, const void* v, const float* g, const float* beta,
                     const float* state_in, float* state_out, void* out,
                     int B, int T, int Hqk, int Hv, int dk, int dv, void* stream);

/*
 * Bytes of device scratch that gdn_prefill needs for the given sizes (host-side
 * arithmetic only; returns 0 for unsupported shapes).  The workspace holds the
 * per-chunk summaries (the chunk table, the cumulative gates, the UT-transformed
 * W and T operands and the masked chunk-local attention matrix).
 */
size_t gdn_prefill_workspace_bytes(int total_tokens, int num_seqs, int Hqk, int Hv, int dk, int dv);

/*
 * Variable-length prefill.  The same recurrence as above, evaluated over 64-token
 * chunks in the chunked WY / UT-transform form (the "chunk-level" reformulation the
 * paper's Sections 3.3 and 5 point to): inside a chunk the triangular system
 * (I + strict_lower(diag(beta) (K K^T o D))) is inverted once, the resulting W and U
 * operands turn the chunk into dense products, and the state is carried serially
 * from chunk to chunk with those products on the tcgen05 tensor cores.
 *
 *   q, k          bf16 [T_tot, Hqk, dk]   sequences packed back to back
 *   v             bf16 [T_tot, Hv, dv]
 *   g, beta       fp32 [T_tot, Hv]
 *   cu_seqlens    int32 [num_seqs+1] on the DEVICE; cu[0] = 0, non-decreasing,
 *                 cu[num_seqs] = total_tokens.  Zero-length sequences are allowed.
 *   initial_state fp32 [num_seqs, Hv, dv, dk] or NULL (all zeros)
 *   out           bf16 [T_tot, Hv, dv]
 *   final_state   fp32 [num_seqs, Hv, dv, dk] or NULL (not wanted); may alias
 *                 initial_state exactly
 *   total_tokens, num_seqs, max_seqlen   host-known sizes (no device sync happens);
 *                 max_seqlen must be >= the longest sequence and <= total_tokens
 *   workspace     >= gdn_prefill_workspace_bytes(...) bytes, 1024-byte aligned
 *
 * Sequences of a batch do not influence each other, whatever their values: a NaN or Inf in
 * one sequence's tokens stays in that sequence's outputs and state.
 *
 * A malformed cu_seqlens can give wrong results but never an out-of-range access:
 * every token index is clamped to [0, total_tokens).  total_tokens = 0 or
 * num_seqs = 0 returns GDN_OK without launching.
 *
 * Few long sequences (num_seqs * Hv chains that would leave most of the GPU idle) are
 * additionally cut into up to 8 runs of chunks that advance at the same time.  The
 * recurrence is affine in the state, S_end = S_in P + H over a run, so each run is
 * walked from the zero state and from the identity, the runs' (P, H) pairs are joined by
 * an associative scan, and the outputs of a run are corrected by S_in (M_t q_t).  This is
 * the same step one level up as the chunked form that Section 5.5 describes (a summary per
 * block of tokens, joined by dense products); the result is the same recurrence, rounded
 * differently.
 * The number of runs follows from num_seqs, Hv and max_seqlen; the environment variable
 * GDN_PREFILL_MAX_SEGMENTS (1..8) lowers it, 1 switches the split off.
 *
 * Many short sequences (more chains than SMs, at most ~10 chunks per sequence on average) are
 * walked by persistent thread blocks, one per SM, that keep their barriers and tensor memory from
 * one chain to the next and fetch the next chain's operands while the current one finishes; what
 * that saves is per chain, so long chains keep one thread block per chain.
 * GDN_PREFILL_PERSISTENT=0/1 in the environment forces one form (same results either way).
 *
 * At the other end, when max_seqlen <= 64 (no sequence longer than one chunk) and a cost model
 * fitted to measurements says the token-serial kernel of gdn_prefill_recurrent is faster (a few
 * short sequences, or many sequences of a handful of tokens), gdn_prefill runs that kernel
 * instead: the narrow short-shape fallback beside a chunked main path that Sections 5.3 and
 * 5.5 mention.  GDN_PREFILL_SHORT_FALLBACK=0 in the environment keeps the chunked kernels.
 * The workspace is required (and checked) either way.
 */
int gdn_prefill(const void* q, const void* k, const void* v, const float* g, const float* beta,
                const int32_t* cu_seqlens, const float* initial_state, void* out, float* final_state,
                int total_tokens, int num_seqs, int max_seqlen,
                int Hqk, int Hv, int dk, int dv,
                void* workspace, size_t workspace_bytes, void* stream);

/*
 * Both entry points with the gate arithmetic fused in (Section 3.2 of the paper, its first
 * two lines): instead of the log-decay g and the write strength beta the caller passes the raw
 * gate inputs
 *   a, b      fp32 [B or T_tot, Hv]     per token and value head
 *   A_log     fp32 [Hv]                 per value head
 *   dt_bias   fp32 [Hv]                 per value head (the paper's b_dt)
 * and the kernels evaluate, in fp32,
 *   alpha = exp(g),  g = -exp(A_log) * softplus(a + dt_bias),   beta = sigmoid(b).
 * All other arguments, results and error behaviour are those of gdn_decode / gdn_prefill.
 */
int gdn_decode_gated(const void* q, const void* k, const void* v, const float* a, const float* b,
                     const float* A_log, const float* dt_bias, const float* state_in, float* state_out, void* out,
                     int B, int Hqk, int Hv, int dk, int dv, void* stream);
int gdn_prefill_gated(const void* q, const void* k, const void* v, const float* a, const float* b,
                      const float* A_log, const float* dt_bias, const int32_t* cu_seqlens,
                      const float* initial_state, void* out, float* final_state,
                      int total_tokens, int num_seqs, int max_seqlen, int Hqk, int Hv, int dk, int dv,
                      void* workspace, size_t workspace_bytes, void* stream);

/*
 * Both entry points with the whole front end of the operator fused in: the raw gates of Section
 * 3.2 as in gdn_decode_gated / gdn_prefill_gated (pass A_log = dt_bias = NULL to give the log-decay g
 * and beta themselves in a and b), and what a layer applies to q and k before the recurrence, which
 * the paper leaves to the caller and this library defines as follows:
 *   qk_l2norm != 0:  q and k of every (token, q/k head) are divided by sqrt(sum of squares + 1e-6),
 *                    the sum over the 128 elements in fp32;
 *   then q is multiplied by `scale` (finite; 1 = none).
 * The kernels do not form normalised copies of q and k: the two per-token factors enter the dot
 * products, the decay coefficients and the output scaling in fp32, so the result is that of the
 * recurrence run on unrounded normalised inputs.  A zero vector stays zero.
 * Errors as for the gated entry points; GDN_ERR_NULL also when exactly one of A_log, dt_bias is NULL;
 * GDN_ERR_SHAPE when scale is not finite.
 */
int gdn_decode_fused(const void* q, const void* k, const void* v, const float* a, const float* b,
                     const float* A_log, const float* dt_bias, const float* state_in, float* state_out, void* out,
                     int B, int Hqk, int Hv, int dk, int dv, float scale, int qk_l2norm, void* stream);
int gdn_prefill_fused(const void* q, const void* k, const void* v, const float* a, const float* b,
                      const float* A_log, const float* dt_bias, const int32_t* cu_seqlens,
                      const float* initial_state, void* out, float* final_state,
                      int total_tokens, int num_seqs, int max_seqlen, int Hqk, int Hv, int dk, int dv,
                      float scale, int qk_l2norm, void* workspace, size_t workspace_bytes, void* stream);
/* gdn_decode_multi (T tokens per item, layouts as there: a, b fp32 [B,T,Hv]) with the same front end. */
int gdn_decode_multi_fused(const void* q, const void* k, const void* v, const float* a, const float* b,
                           const float* A_log, const float* dt_bias, const float* state_in, float* state_out,
                           void* out, int B, int T, int Hqk, int Hv, int dk, int dv,
                           float scale, int qk_l2norm, void* stream);

/*
 * Token-serial prefill: the same inputs and outputs as gdn_prefill (no workspace),
 * computed by the per-token recurrence of Section 3.2 with the state rows held in
 * registers and split along V across thread blocks (the paper's own prefill shape).
 * Kept for very short sequences and as an on-device cross-check of the chunked path.
 */
int gdn_prefill_recurrent(const void* q, const void* k, const void* v, const float* g, const float* beta,
                          const int32_t* cu_seqlens, const float* initial_state, void* out,
                          float* final_state, int total_tokens, int num_seqs, int max_seqlen,
                          int Hqk, int Hv, int dk, int dv, void* stream);

/*
 * Prefill without a caller-provided workspace and without any allocation.  (The paper has no
 * counterpart for this entry point; it exists for integration reasons only.)
 *
 * Who needs it: code that runs where device memory may not be allocated -- a plugin or
 * operator called inside a framework whose memory pool is frozen for the duration of the call,
 * a serving loop that pre-sized all of its buffers at start-up and forbids allocation on the
 * request path, a host that has handed all of its device memory to another allocator.  Such
 * callers can pass inputs and outputs they already own but have nowhere to get the
 * gdn_prefill workspace from.
 *
 * Same arguments and results as gdn_prefill, minus the workspace.  The scratch is a fixed
 * array of GDN_PREFILL_STATIC_SCRATCH_BYTES inside the library image: every device that
 * loads the library holds those bytes until the process exits.  Problems whose workspace
 * (gdn_prefill_workspace_bytes) exceeds that size are refused with GDN_ERR_WORKSPACE; nothing
 * is launched in that case.  The call itself performs no cudaMalloc/cudaFree and calls no
 * allocating library routine.  The kernels see the scratch 1024-byte aligned, like a caller's
 * workspace.
 *
 * Same values, not the same speed: this entry point always runs the chunked kernels with one
 * chain per (sequence, value head).  It never cuts long sequences into runs that advance at
 * the same time (that needs scratch in proportion to the token count) and never hands short
 * sequences to the token-serial kernel, so few long sequences and very short ones run slower
 * here than through gdn_prefill.
 *
 * Device status: pass workspace = NULL to gdn_last_device_status to read (and clear) the
 * status word of this scratch on the current device.
 *
 * The first call on each device looks up the array's device address (with that device
 * current) and remembers it; make that first call outside any stream capture.
 *
 * All calls on a device share the one array, and it keeps whatever the previous call left in
 * it.  Each call rewrites everything it later reads (the chunk table, the status word and
 * every per-chunk block it uses), so stale contents are harmless, but two calls that overlap
 * on the GPU -- different streams, or the same stream from two threads without ordering --
 * race on the scratch and corrupt each other.  Serialise them.
 */
#define GDN_PREFILL_STATIC_SCRATCH_BYTES (32u * 1024u * 1024u)
int gdn_prefill_static(const void* q, const void* k, const void* v, const float* g, const float* beta,
                       const int32_t* cu_seqlens, const float* initial_state, void* out, float* final_state,
                       int total_tokens, int num_seqs, int max_seqlen,
                       int Hqk, int Hv, int dk, int dv, void* stream);

/*
 * Building blocks of sequence-parallel prefill: one long sequence (or each of several) cut into
 * consecutive pieces that are processed at the same time, e.g. one piece per GPU.  The paper
 * evaluates single-GPU kernels only and has no counterpart; the algebra is the recurrence of
 * Section 3.2 written as an affine map of the state.  Over a piece of tokens, with M_t the
 * product of the per-token transitions alpha (I - beta k k^T) from the start of the piece up to
 * token t and H_t the state reached from the zero state,
 *
 *     S_t = S_in M_t + H_t,        o_t = S_t q_t = H_t q_t + S_in (M_t q_t).
 *
 * gdn_prefill_partial   runs a piece without knowing S_in.  Arguments as gdn_prefill, and
 *     out0  bf16 [T_tot, Hv, dv]       H_t q_t (the outputs the zero state would give)
 *     qt    bf16 [T_tot, Hv, dk]       M_t q_t (queries carried back to the start of the piece)
 *     H     fp32 [num_seqs, Hv, dv, dk]   H at the end of each sequence of the piece
 *     P     fp32 [num_seqs, Hv, dk, dk]   M at the end: S_end = S_in P + H
 *     workspace: as gdn_prefill.  An empty sequence gives H = 0, P = I.
 * gdn_state_scan        folds pieces in order: S_out = (...((S0 P_0 + H_0) P_1 + H_1)...), fp32.
 *     P, H  fp32 [steps, num_seqs, Hv, 128, 128] (for instance the all-gathered results of the
 *           pieces before this one); S0 fp32 [num_seqs, Hv, dv, dk] or NULL (zeros);
 *           S_out may alias S0 exactly.  steps = 0 copies S0.
 * gdn_prefill_apply     finishes a piece once its entering state is known:
 *     out[t] += S_in qt[t] for every token (out holds out0 on entry; rounded to bf16 again).
 *     S_in fp32 [num_seqs, Hv, dv, dk]; workspace >= 1024 + num_seqs * Hv * 32768 bytes,
 *     1024-byte aligned (a gdn_prefill workspace for the same sizes is large enough).
 * The state leaving a piece is gdn_state_scan(S_in, P, H, steps = 1).
 * A piece that starts a sequence can instead run gdn_prefill with the known initial state and
 * publish (P, H) = (0, its final state).
 */
int gdn_prefill_partial(const void* q, const void* k, const void* v, const float* g, const float* beta,
                        const int32_t* cu_seqlens, void* out0, void* qt, float* H, float* P,
                        int total_tokens, int num_seqs, int max_seqlen, int Hqk, int Hv, int dk, int dv,
                        void* workspace, size_t workspace_bytes, void* stream);
int gdn_state_scan(const float* S0, const float* P, const float* H, int steps, float* S_out,
                   int num_seqs, int Hv, int dk, int dv, void* stream);
int gdn_prefill_apply(const float* S_in, const void* qt, void* out, const int32_t* cu_seqlens,
                      int total_tokens, int num_seqs, int max_seqlen, int Hv, int dk, int dv,
                      void* workspace, size_t workspace_bytes, void* stream);

/*
 * Reads (and clears) the device-side status word that the prefill kernels set when a
 * bounded wait on an asynchronous copy or tensor-core completion ran out.  HOST
 * pointer out; synchronises `stream`.  *device_status == 0 means no kernel gave up.
 * workspace = NULL reads the fixed scratch of gdn_prefill_static on the current device
 * (GDN_ERR_NULL if gdn_prefill_static has not run on it yet).
 */
int gdn_last_device_status(void* workspace, int* device_status, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* GDN_H_ */
