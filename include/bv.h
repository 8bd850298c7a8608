/*
 * bv.h -- C ABI of the batched draft-verification step of speculative decoding
 * ("Block Verification Accelerates Speculative Decoding", arXiv 2403.10444)
 * for NVIDIA B200 (sm_100a).
 *
 * One call verifies B independent drafted blocks of gamma tokens each.
 *
 * Notation (0-based storage rows, 1-based tokens), T = temperature:
 *   P_r = softmax(target_logits[b, r, :] / T), r = 0..gamma    -- M_b(. | c, X^r)
 *   Q_r = softmax(draft_logits [b, r, :] / T), r = 0..gamma-1  -- M_s(. | c, X^r)
 *   X_i = draft_tokens[b, i-1], i = 1..gamma, drawn from Q_{i-1}
 *   eta_i = uniforms[b, i-1], i = 1..gamma      (acceptance tests)
 *   uniforms[b, gamma]    drives the residual sample (tau < gamma)
 *   uniforms[b, gamma+1]  drives the target sample   (tau = gamma)
 *
 * Layout: every tensor is dense, row-major, contiguous.  dtype selects the
 * logit storage type; all arithmetic is fp32 per element with fp64 combination
 * of partial sums and an fp64 scalar recursion.
 *
 * Sampling is inverse-CDF in vocabulary-index order with weights w_x >= 0,
 * W = sum w, C_k = sum_{x<=k} w_x:  Y = min{k : C_k > u * W}.
 *
 * Ownership: the caller owns every buffer; inputs are never written.  The
 * device entry points enqueue work on `stream` and return without
 * synchronising; buffers must stay valid until that work has completed.
 * The library keeps one workspace per stream (up to 32 streams per device, the
 * least recently used one is recycled beyond that): calls on one stream run in
 * order and share it, calls on different streams never do.  A workspace is
 * obtained and grown with cudaMallocAsync / cudaFreeAsync on that stream, so a
 * first or larger call allocates but does not synchronise the device; the
 * memory is returned by bv_release().  B = 0 is accepted and does nothing.
 *
 * Errors: every entry point returns BV_OK (0) or a negative bv_status; nothing
 * is launched when an argument is rejected.  Data faults are per sequence: a
 * NaN or +inf logit in a row the algorithm reads, a row of all -inf, a drafted
 * token outside [0, V) or whose draft logit is -inf give out_len[b] = -1 and
 * out_tokens[b, :] = -1; other sequences are unaffected.
 */
#ifndef BV_H_
#define BV_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum bv_status {
    BV_OK = 0,
    BV_ERR_INVALID_ARG = -1,  /* null pointer, B < 0, gamma < 1, V < 1, T <= 0 or not finite,
                                 unknown dtype, pointer not aligned to its element size */
    BV_ERR_UNSUPPORTED = -2,  /* gamma > BV_MAX_GAMMA, or no sm_100 device              */
    BV_ERR_CUDA = -3,         /* a CUDA runtime call failed; see bv_last_cuda_error()   */
    BV_ERR_TIMEOUT = -4,      /* a bounded device-side wait gave up: reported by the
                                 host-buffer entry points and by bv_stream_status(),
                                 which synchronise; outputs of that call are invalid   */
    BV_ERR_TOO_LARGE = -5     /* bv_verify_noalloc: B, gamma, V need more scratch than
                                 BV_NOALLOC_SCRATCH_BYTES                               */
} bv_status;

enum { BV_DTYPE_F32 = 0, BV_DTYPE_BF16 = 1 };
enum { BV_MAX_GAMMA = 64 };
enum { BV_NOALLOC_SCRATCH_BYTES = 8 * 1024 * 1024 };

/*
 * Block Verification: Algorithm 2 with Eq. "def_as" (p_0 = 1,
 * p_i = min(p_{i-1} P_{i-1}(X_i)/Q_{i-1}(X_i), 1)), Eq. "pacc_block"
 * (S_i = sum_x max(p_i P_i(x) - Q_i(x), 0); h_gamma = p_gamma,
 * h_i = S_i / (S_i + 1 - p_i), taken as 0 when S_i = 0), tau = the largest i
 * with h_i > 0 and eta_i <= h_i (0 if none), and Y drawn from Eq. "pres-block"
 * at position tau, or from P_gamma when tau = gamma.
 *
 * All pointers are DEVICE pointers.
 *   target_logits [B, gamma+1, V]  dtype      draft_logits [B, gamma, V]  dtype
 *   draft_tokens  [B, gamma]  int32           uniforms     [B, gamma+2]  float in [0,1)
 *   out_tokens    [B, gamma+1] int32: X_1..X_tau, Y, then -1
 *   out_len       [B] int32: tau + 1, or -1 for a sequence with a data fault
 *   stream        a cudaStream_t (NULL = the default stream)
 * Rows whose byte length is a multiple of 16 with 16-byte aligned bases use the
 * 128-bit path; any other V >= 1 is served by an element-wise path.
 * Since S_i <= p_i, h_i <= p_i: on the 128-bit path S_i is evaluated only for
 * positions with eta_i <= p_i, from the highest down to the first one that passes
 * eta_i <= h_i; tau and Y are those of the full evaluation (bv_verify_ex does the
 * full evaluation).  The cost of a call therefore depends on how many drafted
 * tokens are accepted.
 */
int bv_verify(const void* target_logits, const void* draft_logits,
              const int32_t* draft_tokens, const float* uniforms,
              int B, int gamma, int V, int dtype, float temperature,
              int32_t* out_tokens, int32_t* out_len, void* stream);

/*
 * Token Verification: Algorithm 1 with Eq. "accept_probability"
 * (h_i = min(P_{i-1}(X_i)/Q_{i-1}(X_i), 1)); tau = length of the initial run of
 * i with h_i > 0 and eta_i <= h_i; Y from Eq. "pres-token" at position tau, or
 * from P_gamma when tau = gamma.  Only rows 0..tau are read.  Arguments as for
 * bv_verify.
 */
int tv_verify(const void* target_logits, const void* draft_logits,
              const int32_t* draft_tokens, const float* uniforms,
              int B, int gamma, int V, int dtype, float temperature,
              int32_t* out_tokens, int32_t* out_len, void* stream);

/*
 * The same two procedures, also writing their intermediates (device pointers,
 * float, any of which may be NULL):
 *   out_p     [B, gamma+1]  p_0..p_gamma                (Eq. "def_as"; NaN for tv)
 *   out_S     [B, gamma]    S_0..S_{gamma-1}            (tv: only S_tau, NaN elsewhere)
 *   out_h     [B, gamma+1]  h_0 := 1, h_1..h_gamma      (tv: up to the first rejection)
 *   out_lse_t [B, gamma+1]  ln sum_x exp(target/T) per row (NaN for rows not read)
 *   out_lse_d [B, gamma]    ln sum_x exp(draft/T)  per row
 */
int bv_verify_ex(const void* target_logits, const void* draft_logits,
                 const int32_t* draft_tokens, const float* uniforms,
                 int B, int gamma, int V, int dtype, float temperature,
                 int32_t* out_tokens, int32_t* out_len,
                 float* out_p, float* out_S, float* out_h,
                 float* out_lse_t, float* out_lse_d, void* stream);
int tv_verify_ex(const void* target_logits, const void* draft_logits,
                 const int32_t* draft_tokens, const float* uniforms,
                 int B, int gamma, int V, int dtype, float temperature,
                 int32_t* out_tokens, int32_t* out_len,
                 float* out_p, float* out_S, float* out_h,
                 float* out_lse_t, float* out_lse_d, void* stream);

/*
 * Host-buffer forms of Algorithm 2 / Algorithm 1: every pointer is a HOST
 * pointer (pinned memory makes the copies asynchronous).  The call copies the
 * inputs to device staging buffers owned by the library (grown on demand, kept
 * until bv_release()), runs the device path on the current device, copies
 * out_tokens and out_len back, and returns after they have landed.
 */
int bv_verify_host(const void* target_logits, const void* draft_logits,
                   const int32_t* draft_tokens, const float* uniforms,
                   int B, int gamma, int V, int dtype, float temperature,
                   int32_t* out_tokens, int32_t* out_len);
int tv_verify_host(const void* target_logits, const void* draft_logits,
                   const int32_t* draft_tokens, const float* uniforms,
                   int B, int gamma, int V, int dtype, float temperature,
                   int32_t* out_tokens, int32_t* out_len);

/*
 * Block Verification without any allocation.  (The paper has no counterpart: this entry
 * point exists for the way the library is embedded, not for the method.)
 *
 * For callers that cannot let a library call cudaMalloc when they call it: servers whose
 * memory pool owns the whole device, code that may run under stream capture, processes
 * with allocator hooks.  Same arguments, outputs and arithmetic as bv_verify(), DEVICE
 * pointers, asynchronous on `stream`; it never calls cudaMalloc, cudaFree or any routine
 * that allocates.  Its scratch is a fixed array of BV_NOALLOC_SCRATCH_BYTES (8 MiB) inside
 * the library image, present on every GPU that loads the library until the process exits.
 *
 * Limits and rules that bv_verify() does not have:
 *   - the scratch needed grows with B (gamma+1), about 2.1 KB per logit row pair at large V
 *     (B = 256, gamma = 8, V = 256000 needs 5.0 MB); a problem that needs more than the
 *     array returns BV_ERR_TOO_LARGE and launches nothing;
 *   - rows must be whole 16-byte vectors on 16-byte aligned bases (V a multiple of 8 for
 *     bf16, of 4 for fp32), else BV_ERR_UNSUPPORTED;
 *   - the first call on each device and for each dtype looks the array's device address up
 *     and queries the device and the kernel's occupancy; make those calls before any stream
 *     capture begins;
 *   - every call on a device uses the same array, which keeps the previous call's contents
 *     (the entry point clears the part that must start at zero, on `stream`).  Two calls
 *     that overlap on the GPU, on different streams, race on it: order them yourself;
 *   - a device-side wait that gives up is not reported (bv_stream_status() does not see this
 *     entry point's calls); the outputs of such a call are left unwritten.
 */
int bv_verify_noalloc(const void* target_logits, const void* draft_logits,
                      const int32_t* draft_tokens, const float* uniforms,
                      int B, int gamma, int V, int dtype, float temperature,
                      int32_t* out_tokens, int32_t* out_len, void* stream);

/*
 * Block Verification with the draft rows' log-normalisers supplied:
 *   draft_lse [B, gamma] float, DEVICE: ln sum_x exp(draft_logits[b, r, x] / temperature),
 *   as bv_sample_draft() leaves them when the drafting step runs through this library.
 * The draft distributions of Algorithm 2 are then M_s(x | c, X^r) = exp(z_x / T - draft_lse[b, r]),
 * and the first sweep does not read the draft rows at all: they are read only for the few positions
 * whose residual mass S_r (Eq. "pacc_block") is needed, so a call moves about half the bytes of
 * bv_verify().  A float normaliser carries about 2e-6 relative error into M_s; the emitted tokens
 * keep the target model's law to that accuracy.  A draft_lse entry that is not finite is a data
 * fault of its sequence (out_len = -1); the contents of a draft row are otherwise trusted.
 * Only the 128-bit path exists (rows of whole 16-byte vectors on 16-byte aligned bases), else
 * BV_ERR_UNSUPPORTED.  Other arguments, outputs and diagnostics as bv_verify / bv_verify_ex
 * (out_lse_d returns the supplied values).
 */
int bv_verify_lse(const void* target_logits, const void* draft_logits,
                  const int32_t* draft_tokens, const float* uniforms, const float* draft_lse,
                  int B, int gamma, int V, int dtype, float temperature,
                  int32_t* out_tokens, int32_t* out_len, void* stream);
int bv_verify_lse_ex(const void* target_logits, const void* draft_logits,
                     const int32_t* draft_tokens, const float* uniforms, const float* draft_lse,
                     int B, int gamma, int V, int dtype, float temperature,
                     int32_t* out_tokens, int32_t* out_len,
                     float* out_p, float* out_S, float* out_h,
                     float* out_lse_t, float* out_lse_d, void* stream);

/*
 * Token Verification (Algorithm 1) with the draft rows' log-normalisers supplied, as bv_verify_lse: the
 * acceptance tests read the target rows only (the draft row of a test contributes the one logit of
 * its drafted token), and a draft row is read in full only where the residual of Eq. "pres-token" is
 * sampled.  Same rules as bv_verify_lse; a draft_lse entry that is not finite counts as a data fault if
 * its row is among rows 0 .. min(tau, gamma - 1).
 */
int tv_verify_lse(const void* target_logits, const void* draft_logits,
                  const int32_t* draft_tokens, const float* uniforms, const float* draft_lse,
                  int B, int gamma, int V, int dtype, float temperature,
                  int32_t* out_tokens, int32_t* out_len, void* stream);
int tv_verify_lse_ex(const void* target_logits, const void* draft_logits,
                     const int32_t* draft_tokens, const float* uniforms, const float* draft_lse,
                     int B, int gamma, int V, int dtype, float temperature,
                     int32_t* out_tokens, int32_t* out_len,
                     float* out_p, float* out_S, float* out_h,
                     float* out_lse_t, float* out_lse_d, void* stream);

/*
 * Greedy Block Verification, one iteration: Algorithm 4.  The running product is not clipped,
 *   pt_0 = 1,  pt_i = pt_{i-1} P_{i-1}(X_i) / Q_{i-1}(X_i);
 * position 0 < i < gamma passes its test when eta_i <= h_i with
 *   h_i = sum_x max(pt_i P_i(x) - Q_i(x), 0) / sum_x max(Q_i(x) - pt_i P_i(x), 0)
 * (the second sum equals the first plus 1 - pt_i; a test with an empty first sum never passes),
 * position gamma when eta_gamma <= pt_gamma (printed with "<"; taken as "<=" like every other
 * test); tau is the highest position that passes (0 if none) and Y is drawn from Eq. "pres_greedy"
 * at position tau (Eq. "pres-block" with pt_tau in place of p_tau), or from P_gamma when tau = gamma.
 * The paper shows that the tokens after (X^tau, Y) must then be drawn from the modified model of
 * Algorithm 5 to keep the target model's law; that step needs the models and is the caller's.
 *
 * Arguments, outputs, errors and uniform usage as bv_verify / bv_verify_ex; DEVICE pointers.
 * Diagnostics: out_p holds pt_0..pt_gamma, out_S the first sums (i = 0..gamma-1), out_h the ratios
 * h_i (h_0 := 1, h_gamma := pt_gamma); a ratio above one is only known to be above one (its
 * denominator is a difference of nearly equal numbers) and is +inf when that denominator is not
 * positive.  As for bv_verify, the sums are evaluated only for positions that can be selected
 * (eta_i <= pt_i) unless diagnostics are asked for.  Only the 128-bit path exists (rows of whole
 * 16-byte vectors on 16-byte aligned bases), else BV_ERR_UNSUPPORTED.
 * The product pt_i is carried in double and handed to the sweeps scaled as a float; a product
 * beyond about 1e38 is outside the supported range (under the draft model E[pt_i] <= 1, so by
 * Markov's inequality that has probability below 1e-38).
 */
int gbv_verify(const void* target_logits, const void* draft_logits,
               const int32_t* draft_tokens, const float* uniforms,
               int B, int gamma, int V, int dtype, float temperature,
               int32_t* out_tokens, int32_t* out_len, void* stream);
int gbv_verify_ex(const void* target_logits, const void* draft_logits,
                  const int32_t* draft_tokens, const float* uniforms,
                  int B, int gamma, int V, int dtype, float temperature,
                  int32_t* out_tokens, int32_t* out_len,
                  float* out_p, float* out_S, float* out_h,
                  float* out_lse_t, float* out_lse_d, void* stream);

/*
 * Algorithms 2 and 1 on given probabilities, the form in which the paper states them (Algorithm 1,
 * Algorithm 2: the conditional distributions M_b(. | c, X^i), M_s(. | c, X^i) are the inputs):
 *   target_probs [B, gamma+1, V], draft_probs [B, gamma, V] in `dtype`, device pointers, 16-byte
 *   aligned, rows of a multiple of 16 bytes (else BV_ERR_UNSUPPORTED); the other arguments as bv_verify.
 * The numbers are used as stored: Eq. "def_as", "pacc_block", "pres-block" / "pres-token" are
 * evaluated on them without renormalising (the samples divide by the sum of their own weights), and
 * no temperature applies.  Only the rows the algorithm needs are read: the 2 gamma entries of the
 * drafted tokens, the row pairs of the positions that can be the selected one (Algorithm 2: those
 * with eta_i <= p_i, from the top down; Algorithm 1: the one at tau), or row gamma of the target.
 * A sequence with a drafted token outside [0, V), with Q_{i-1}(X_i) not a positive finite number or
 * P_{i-1}(X_i) not a non-negative finite number (Algorithm 1: in a test it makes), or with an empty
 * or non-finite weight sum where it must sample, gets out_len = -1 and out_tokens = -1; entries the
 * algorithm does not read are not validated.
 * out_p [B, gamma+1], out_S [B, gamma], out_h [B, gamma+1]: optional diagnostics as in bv_verify_ex /
 * tv_verify_ex (each may be null; with any of them Algorithm 2 evaluates every position).
 */
int bv_verify_probs(const void* target_probs, const void* draft_probs,
                    const int32_t* draft_tokens, const float* uniforms,
                    int B, int gamma, int V, int dtype,
                    int32_t* out_tokens, int32_t* out_len,
                    float* out_p, float* out_S, float* out_h, void* stream);
int tv_verify_probs(const void* target_probs, const void* draft_probs,
                    const int32_t* draft_tokens, const float* uniforms,
                    int B, int gamma, int V, int dtype,
                    int32_t* out_tokens, int32_t* out_len,
                    float* out_p, float* out_S, float* out_h, void* stream);

/*
 * The drafting step of Algorithm 3 (its first step: one token per draft distribution, the
 * distribution's normaliser kept for the verification) for `rows` rows of draft logits [rows, V]:
 *   out_tokens[r] ~ softmax(logits[r, :] / temperature), drawn by inverse CDF in vocabulary-index
 *                   order with uniforms[r] in [0, 1): min{k : C_k > u W} over the running sums C_k of
 *                   the weights, the convention of the verification samples;
 *   out_lse[r]    = ln sum_x exp(logits[r, x] / temperature)  (float; may be NULL).
 * DEVICE pointers, asynchronous on `stream`, no allocation.  A row with a NaN or +inf logit, or
 * with no finite logit, gives out_tokens[r] = -1 and out_lse[r] = NaN.  Rows must be whole 16-byte
 * vectors on a 16-byte aligned base (V a multiple of 8 for bf16, of 4 for fp32), else
 * BV_ERR_UNSUPPORTED.  Each logit is read from HBM once.
 */
int bv_sample_draft(const void* logits, const float* uniforms, int rows, int V, int dtype,
                    float temperature, int32_t* out_tokens, float* out_lse, void* stream);

/*
 * The drafting step of Algorithm 3 as a whole for a draft model whose next-token logits depend on the
 * last token only: draft_table [V, V] in `dtype`, DEVICE, row t = the logits after token t.  For each
 * of B sequences, starting from first_tokens[b] (int32, DEVICE), gamma tokens are drawn one after the
 * other, X_{i+1} from softmax(draft_table[X_i, :] / temperature) by the convention of
 * bv_sample_draft with uniforms[i, b] (uniforms [gamma, B] float, DEVICE):
 *   out_tokens [B, gamma] int32, out_lse [B, gamma] float (may be null): the tokens and the
 *   log-normalisers of the rows they were drawn from, as bv_verify_lse / tv_verify_lse take them.
 * One launch instead of gamma dependent ones.  A first token outside [0, V) or a row that cannot be
 * sampled (see bv_sample_draft) ends that sequence's chain: its remaining tokens are -1, their
 * normalisers NaN.  Rows must be whole 16-byte vectors on a 16-byte aligned base, else BV_ERR_UNSUPPORTED.
 */
int bv_draft_chain(const void* draft_table, const int32_t* first_tokens, const float* uniforms,
                   int B, int gamma, int V, int dtype, float temperature,
                   int32_t* out_tokens, float* out_lse, void* stream);

/*
 * Waits for `stream` and reports whether a device-side wait of any call enqueued on it since the
 * last query gave up: BV_ERR_TIMEOUT (the outputs of those calls are not to be used; the library's
 * state is intact and later calls work) or BV_OK.  Every device-side wait of this library is
 * bounded, so a protocol error ends a kernel instead of hanging the GPU; this call is how a user
 * of the device entry points learns of it.  The host-buffer entry points do the same themselves.
 */
int bv_stream_status(void* stream);

/*
 * Tuning and test options, process-wide, read by every later call (0 restores the default choice):
 *   "kernel"        1 flow, 2 cluster, 3 element-wise streaming kernel, 4 small-batch kernel (for the shapes
 *                   each admits; the default picks the small-batch kernel for up to 32 sequences whose
 *                   logits are few enough to make the launch a matter of latency - up to 16 sequences for
 *                   the entry points on probabilities -, else the flow kernel)
 *   "small_bytes"   logit megabytes up to which the small-batch kernel is the default
 *   "cluster"       cluster width of the cluster / streaming kernels (1, 2, 4, 8)
 *   "max_clusters"  cap on the clusters those kernels launch
 *   "flow_chunks", "flow_pieces", "flow_ctas", "flow_depth"   work-item shape of the flow kernel (chunks per row in
 *                   the first sweep, pieces per row in the second, CTAs launched, descriptors a CTA hands to its
 *                   workers ahead of the sweep: 2 for Block Verification, 3 for Algorithm 1 and with diagnostic outputs)
 *   "flow_keep_l2"  1: the lines a first sweep loads stay in L2 at normal priority for the row's second
 *                   sweep (default 0: every load of the flow kernel streams past L2, which measured faster)
 *   "flow_fine"     n > 0: Block Verification cuts the rows of the last n sequences of the batch into the finer
 *                   chunks that last target rows get, so that the launch ends on short items (default 0:
 *                   none; it helped only where most drafted tokens are accepted)
 *   "wait_limit"    polls after which a bounded device-side wait gives up (tests)
 *   "never_signal"  tests: the flow kernel's workers never report an item as swept, so its waits
 *                   run out and the call ends with BV_ERR_TIMEOUT
 * Their first values come from the environment variables BV_KERNEL (flow / cluster / stream / small),
 * BV_CLUSTER, BV_MAX_CLUSTERS, BV_FLOW_CHUNKS, BV_FLOW_PIECES, BV_FLOW_CTAS, BV_FLOW_DEPTH, read once.
 * Returns BV_ERR_INVALID_ARG for an unknown name.
 */
int bv_set_option(const char* name, int value);

/* Frees the library's cached device buffers on the current device (waits for the device). */
int bv_release(void);

/* Number of kernel launches the last device-path call on this thread enqueued. */
int bv_last_launch_count(void);
/* Which kernel the last bv_verify / tv_verify (or _ex, _lse, _probs, gbv_, _host) call on this thread launched, in the
 * codes of the "kernel" option: 1 flow, 2 cluster, 3 element-wise streaming, 4 small-batch; 0 if it launched none. */
int bv_last_kernel(void);
/* cudaError_t value of the last failing runtime call on this thread (0 if none). */
int bv_last_cuda_error(void);
/* Static description of a bv_status value. */
const char* bv_status_string(int status);
/* Library version: major * 10000 + minor * 100 + patch. */
int bv_version(void);

#ifdef __cplusplus
}
#endif
#endif /* BV_H_ */
