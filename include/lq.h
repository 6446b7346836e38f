/*
 * liblq: layer-wise unbiased stochastic quantization and the Quantized Optimistic Dual
 * Averaging (QODA) update for K data-parallel workers simulated on one GPU.
 *
 * Conventions
 *  - Every function returns an int: LQ_OK (0) or a negative LQ_E* code.  Nothing throws,
 *    aborts or traps.  lq_last_error() gives a human-readable reason for the calling
 *    thread's last failure.
 *  - "dev" pointers are device memory OWNED BY THE CALLER (allocated however the caller
 *    likes); "host" pointers are ordinary host memory.  The plan owns only its own
 *    tables and scratch, released by lq_plan_destroy.
 *  - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Calls that
 *    take a stream only enqueue work on it and return; they do not synchronise unless
 *    stated.  Calls on one plan must be issued in stream order by the caller.
 *  - fp32 rows (grads, X1, Y, Xhalf, X, gbar) must start on a 16-byte boundary, message and norm
 *    buffers on a 4-byte boundary; a misaligned pointer is refused with LQ_EINVAL.
 *  - Argument errors are reported synchronously.  Data problems (NaN/Inf input, zero
 *    norm) never fault: they set per-(worker, layer) status flags, see lq_get_statistics.
 *
 * Data layout
 *  - A plan is a ragged list of L layers with sizes d_m, code widths b_m (n_m = 2^b_m levels
 *    per layer, including 0 and 1), one norm order q, K workers and a 64-bit seed.
 *  - Gradient-like buffers (grads, X1, Y, Xhalf, X, gbar) are fp32 rows of D_pad =
 *    lq_plan_padded_elems() elements; layer m starts at element elem_off_m (a multiple of 32)
 *    and its d_m values are contiguous.  grads is [K][D_pad], row-major.  Elements between
 *    layers are padding: never interpreted on input, may be overwritten on output.
 *  - A worker's message is W = lq_plan_packed_words() 32-bit words; packed is [K][W].
 *    Every coordinate becomes one symbol of b+1 bits, symbol = 2 * level index + sign.
 *    Layer m starts at word_off_m and is cut into blocks of 1024 coordinates (the last one
 *    zero-padded).  A block is (b+1) planes of 32 words.  Coordinate c of a block belongs to
 *    lane (c/4)%32 and has position p = 4*(c/128) + c%4 in that lane.  The 32 symbols of a lane
 *    form one little-endian string of 32*(b+1) bits with symbol p at bit offset p*(b+1); bit t
 *    of that string is bit t%32 of word (t/32)*32 + lane of the block.
 *    The norms travel separately as fp32: norms is [K][L].
 *    (Section 3.2 of the paper fixes the content of a message: a 32-bit float norm, one sign
 *    bit and one integer code per coordinate; the physical arrangement is this library's.)
 */
#ifndef LQ_H_
#define LQ_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define LQ_OK       0
#define LQ_EINVAL  (-1)   /* bad argument (NULL, size, range, non-increasing levels, ...) */
#define LQ_ENOMEM  (-2)   /* host or device allocation failed */
#define LQ_ECUDA   (-3)   /* a CUDA runtime call failed; see lq_last_error() */
#define LQ_ESTATE  (-4)   /* call out of order (e.g. qoda_step before qoda_init) */

#define LQ_NUM_BINS     386   /* histogram bins per (worker, layer) */
#define LQ_HIST_STRIDE  512   /* words between consecutive histograms */
#define LQ_MAX_BITS     8
#define LQ_MAX_WORKERS  1024

#define LQ_STATUS_ZERO_NORM  1u  /* layer norm below the smallest normal float: message is all zero */
#define LQ_STATUS_NONFINITE  2u  /* NaN/Inf in the layer (or norm overflow): message is all zero, norm 0 */

typedef struct lq_plan lq_plan;

/* Plan over a ragged list of layers (Section 3.1: each layer follows its own sequence of
 * levels; Section 2.2: L^q normalisation).
 *   layer_sizes [num_layers] host, each in [0, 2^31);  bits [num_layers] host, each in [1, 8];
 *   q >= 1 is the norm order (1..16), q = 0 selects the infinity norm;
 *   num_workers in [1, LQ_MAX_WORKERS];  seed keys the Philox4x32-10 stream together with
 *   (step, worker, layer, coordinate).
 * Every layer starts with uniform levels j/(2^b-1).  Allocates device tables and scratch on
 * the current device; may synchronise.  On failure *out is NULL. */
int lq_plan_create(lq_plan** out, int32_t num_layers, const int64_t* layer_sizes,
                   const int32_t* bits, int32_t q, int32_t num_workers, uint64_t seed);
int lq_plan_destroy(lq_plan* plan);             /* synchronises the device; NULL is accepted */

int64_t lq_plan_padded_elems(const lq_plan* plan);   /* D_pad, or LQ_EINVAL */
int64_t lq_plan_packed_words(const lq_plan* plan);   /* W, or LQ_EINVAL */
/* Any of the three outputs may be NULL. */
int lq_plan_layer_info(const lq_plan* plan, int32_t layer, int64_t* elem_off, int64_t* word_off,
                       int32_t* num_levels);

/* Norm scope.  LQ_NORM_PER_LAYER (default): every layer is normalised by its own L^q norm.
 * LQ_NORM_GLOBAL: the formal definition of Q in Section 3.1 - one norm ||v||_q over the worker's whole vector
 * (all layers), per-layer level sequences; norms[k][m] then holds that one value for every m, so messages
 * and every other call keep their format.  A NaN or Inf anywhere then zeroes the worker's whole message.
 * Takes effect at the next lq_layer_norms / lq_quantize_pack. */
#define LQ_NORM_PER_LAYER 0
#define LQ_NORM_GLOBAL    1
/* LQ_NORM_BUCKET: the setting of the experiments in Section 7.1 - every bucket of LQ_BUCKET = 128 consecutive
 * coordinates of a layer (the last one of a layer may be shorter) is normalised by its own L^q norm, with the
 * layer's level sequence.  Differences from the other scopes:
 *  - a norms buffer is [K][lq_plan_norm_count()] fp32: for layer m, block i of 1024 coordinates and row j of 128,
 *    the bucket's norm sits at 8 * (blocks of the layers before m + i) + j; rows past the layer's end hold 0.
 *    lq_quantize_pack WRITES it in its single pass over the values (there is no separate norm pass and
 *    lq_layer_norms is refused); prev_norms, lq_decode_aggregate and qoda_step read the same shape;
 *  - a bucket that is all zero, whose norm is below the smallest normal float, or that holds NaN or Inf has norm
 *    0 and sends zeros; the layer's flag (lq_get_statistics) is LQ_STATUS_NONFINITE if any of its buckets held NaN
 *    or Inf, else LQ_STATUS_ZERO_NORM if none of its buckets has a nonzero norm;
 *  - the histogram of a (worker, layer) pools its buckets' normalised magnitudes (zeroed buckets add nothing);
 *    lq_fit_levels, lq_fit_levels_shared and lq_level_probabilities weight worker k's histogram of layer m by
 *    the layer's energy, the sum of its squared bucket norms as left by the plan's last lq_quantize_pack
 *    (lq_layer_weights returns its square root), and do not read their `norms` argument (any non-NULL pointer).
 * The bucket scope can only be entered or left before the plan's first lq_quantize_pack (else LQ_ESTATE). */
#define LQ_NORM_BUCKET    2
#define LQ_BUCKET         128
int lq_set_norm_scope(lq_plan* plan, int32_t scope);
/* Worker range (several processes sharing one job: Algorithm 1 has every node encode its own dual vector and
 * broadcast it).  After lq_set_worker_range(plan, first, count) the encode-side calls - lq_layer_norms and
 * lq_quantize_pack - handle only workers first .. first + count - 1: `grads` is [count][D_pad] (row 0 = worker
 * `first`), while packed, norms, hist, prev_packed and prev_norms keep their full [K] shapes and only the rows of
 * the range are read or written; the random numbers are those of the workers' global indices, so K processes of
 * one worker each emit the same messages as one process of K workers.  The caller then brings the other workers'
 * rows of packed and norms in (an all-gather), and their per-(worker, layer) side data - the step-size statistic
 * that qoda_step consumes, the bucket scope's fit weights, the flags - with the two calls below, before
 * lq_decode_aggregate / qoda_step / lq_fit_levels, which always cover all K workers.  Default range: (0, K).
 * A plan keeps track of one stream of messages (level tables and zero-row masks of the previous one), so choose
 * the range once, before the first lq_quantize_pack; after a later change the next lq_quantize_pack must start a
 * new stream (prev_packed = NULL, else LQ_ESTATE).  LQ_EINVAL if the range does not lie inside [0, K). */
int lq_set_worker_range(lq_plan* plan, int32_t first_worker, int32_t count);
/* Copies the plan's per-(worker, layer) side data to / from DEVICE arrays of shape [K][L] on `stream`
 * (sq_diff fp64, 8-byte aligned; layer_weight fp32; flags u32; any pointer may be NULL = skip).  Export after
 * lq_quantize_pack, exchange the rows, import before qoda_step. */
int lq_side_data_export(const lq_plan* plan, double* sq_diff, float* layer_weight, uint32_t* flags, void* stream);
int lq_side_data_import(lq_plan* plan, const double* sq_diff, const float* layer_weight, const uint32_t* flags,
                        void* stream);

/* fp32 values per worker in a norms buffer under the plan's current scope: the number of layers, or in bucket
 * scope 8 x the number of 1024-coordinate blocks of all layers.  Negative error code on failure. */
int64_t lq_plan_norm_count(const lq_plan* plan);
/* Bucket scope: host_weights [K][L] receives sqrt(sum of squared bucket norms) of every (worker, layer) of the
 * plan's last lq_quantize_pack.  Synchronises the device.  LQ_ESTATE in another scope. */
int lq_layer_weights(const lq_plan* plan, float* host_weights);

/* Level sequence of one layer (Section 3.1: 0 = l_0 < l_1 < ... < l_{n-1} = 1, n = 2^b).
 * host_levels [n] host.  set: validates (n must equal 2^b, increasing by at least 2^-100 per
 * step, ends 0 and 1)
 * and stages the sequence; it is used from the next lq_quantize_pack on.  get: returns the
 * staged sequence (the most recent of set / fit).  Both synchronise the device. */
int lq_set_levels(lq_plan* plan, int32_t layer, const float* host_levels, int32_t n);
int lq_get_levels(const lq_plan* plan, int32_t layer, float* host_levels, int32_t n);

/* Per-layer L^q norms only (Section 2.2): norms[k][m] = fp32(||grads[k][layer m]||_q),
 * accumulated in fp64.  grads dev [K][D_pad]; norms dev [K][L].  Updates the status flags. */
int lq_layer_norms(lq_plan* plan, const float* grads, float* norms, void* stream);

/* ENCODE for all K workers (Algorithm 1 line 12; Section 3.1 quantizer, Section 3.2 message):
 * per-layer norm, normalisation u = min(|v| * (1/N), 1), stochastic rounding of u between its
 * two neighbouring levels (up with probability (u - l_tau)/(l_{tau+1} - l_tau), uniforms from
 * Philox keyed (seed, step, worker, layer, coordinate)), sign and index packing.
 *   grads dev [K][D_pad];  packed dev [K][W] (fully overwritten);  norms dev [K][L] out;
 *   hist: NULL, or dev [K][L][LQ_HIST_STRIDE] u32 histograms of u, ADDED to (caller zeroes
 *     them); bin 0 = [0,2^-24), then 16 bins per octave up to 1, bin 385 = {1}
 *     (Algorithm 1 line 4);
 *   prev_packed / prev_norms: the message this plan produced in its previous
 *     lq_quantize_pack call (dev [K][W], [K][L]), or both NULL when there is none
 *     (V^_{k,1/2} = 0).  Used for the step-size statistic
 *     sum_k ||V^_{k,t+1/2} - V^_{k,t-1/2}||^2 of Eq. (general_stepsize), which is left
 *     inside the plan for the next qoda_step: per coordinate the fp32 difference of the two
 *     decoded fp32 values, its square summed in fp64.  The previous message is decoded with the
 *     levels it was encoded with, even if the levels were changed in between.  It must hold the
 *     message of this plan's previous lq_quantize_pack call (that message's levels and norms
 *     decode it).  When it is the very buffer that call wrote, the plan uses what it remembers of
 *     that call - which rows of its input were all zero - and does not read the corresponding
 *     words again; a copy at another address is read in full.  A caller that rewrote the buffer
 *     in place says so with lq_message_modified.
 *   prev_packed must not alias packed.
 *   The sign of a coordinate is (v < 0): +0 and -0 both give symbol 0, so rows of zeros (of either
 *   sign) become all-zero words; such rows are detected by the norm pass and not read again.
 *   step = LQ_STEP_AUTO: the kernels take the step index from the plan's iteration counter on the device (the
 *   t of qoda_get_scalars, advanced by every qoda_step, 1 after qoda_init) instead of from the host.  Then no
 *   argument of an iteration changes from one pair of iterations to the next, so a caller may record
 *   [lq_quantize_pack, qoda_step] x 2 (two iterations, because messages and masks are double-buffered) into a
 *   CUDA graph on its stream and replay it: every call only enqueues work on `stream` and keeps its plan-side
 *   bookkeeping on the host, where the replays leave it as the recording did.  A level change (lq_set_levels,
 *   lq_fit_levels) needs a new recording, and profiling (lq_profile_enable) must be off while recording. */
#define LQ_STEP_AUTO 0xFFFFFFFFu
int lq_quantize_pack(lq_plan* plan, const float* grads, uint32_t step, uint32_t* packed,
                     float* norms, uint32_t* hist, const uint32_t* prev_packed,
                     const float* prev_norms, void* stream);

/* Level update (Algorithm 1 lines 2-7; Section 3.2, the minimisation after Eq. MQV with the
 * CDF weights lambda_z = N_z^2 / sum N_z^2): for every layer with at least 3 levels, merge
 * the num_samples histograms of that layer with those weights and minimise
 * sum_j int_{l_j}^{l_{j+1}} (l_{j+1}-u)(u-l_j) dF~(u) by exact coordinate minimisation
 * (the solver is this library's: the paper states the objective only).  The descent runs from two
 * starts, the quantiles of the merged mass and the uniform grid, and the end point with the smaller
 * objective is kept; the result is a stationary point, for a density that is not log-concave not
 * necessarily the global minimum.
 *   hist dev [num_samples][L][LQ_HIST_STRIDE];  norms dev [num_samples][L].
 * The new levels are staged: they take effect at the next lq_quantize_pack.  Layers with no
 * usable mass keep their levels. */
int lq_fit_levels(lq_plan* plan, const uint32_t* hist, const float* norms, int32_t num_samples,
                  void* stream);

/* Level update with one sequence per TYPE (Section 3.1: the coordinates are split into M types, each with
 * its own sequence; a type here is a set of layers).  layer_type host [L]: layers with equal ids form a type and
 * must have the same code width.  The histograms of all (sample, member layer) pairs of a type are merged with
 * weights N^2 - the variance being minimised is sum N_s^2 sum_i sigma_Q^2(u_i) - and every member receives the
 * fitted sequence (staged, like lq_fit_levels; with every layer a type of its own the result is that of
 * lq_fit_levels up to rounding).  hist, norms, num_samples as for lq_fit_levels.  The id list is copied
 * before the call returns. */
int lq_fit_levels_shared(lq_plan* plan, const uint32_t* hist, const float* norms, int32_t num_samples,
                         const int32_t* layer_type, void* stream);

/* DECODE + aggregate (Algorithm 1 lines 15 and 17): gbar = (1/K) sum_k N_k * sign * l_idx,
 * summed in fp32 in worker order, with the levels of the latest lq_quantize_pack.
 *   packed dev [K][W];  norms dev [K][L];  gbar dev [D_pad] out. */
int lq_decode_aggregate(const lq_plan* plan, const uint32_t* packed, const float* norms,
                        float* gbar, void* stream);

/* QODA state (Algorithm 1; Eq. ODA).  qoda_init sets Y_1 = 0, X_{3/2} = X_1, S_0 = 0,
 * eta_1 = 1, t = 1 (initialisation V^_{k,1/2} = 0).   X1, Y, Xhalf dev [D_pad]. */
int qoda_init(lq_plan* plan, const float* X1, float* Y, float* Xhalf, void* stream);

/* One QODA iteration after the workers' messages exist (Algorithm 1 lines 15-18 and line 10
 * of the next iteration; Eq. ODA; Eq. general_stepsize):
 *   S_t = S_{t-1} + (statistic left by the last lq_quantize_pack) / K^2,
 *   eta_{t+1} = gamma_{t+1} = fp32((1 + S_t)^(-1/2)),
 *   gbar = mean of the K decoded messages,  Y_{t+1} = Y_t - gbar,
 *   X_{t+1} = fma(eta_{t+1}, Y_{t+1}, X_1),  X_{t+3/2} = fma(-gamma_{t+1}, gbar, X_{t+1}).
 * One fused pass: each packed message is read once.
 * qoda_step consumes the message of the plan's last lq_quantize_pack (whose statistic it uses; LQ_ESTATE if there
 * is no new one).  When `packed` is the very buffer that call wrote for all K workers (layer or global scope),
 * the buffer must still hold that message: blocks the encoder knows to be all zero are not read again, and where no
 * worker sent anything Y is left as it is.  A message at another address, and one assembled from several worker
 * ranges, is read in full; so is that buffer after lq_message_modified, the call by which a caller who has
 * rewritten the buffer in place (its own exchange, say) tells the plan that what it remembers of the last
 * lq_quantize_pack's input no longer describes the words there.  The next lq_quantize_pack starts afresh.
 *   packed dev [K][W], norms dev [K][L], X1 dev [D_pad] in;  Y dev [D_pad] in/out;
 *   Xhalf dev [D_pad] out (X_{t+3/2});  X_opt, gbar_opt: NULL or dev [D_pad] out. */
int qoda_step(lq_plan* plan, const uint32_t* packed, const float* norms, const float* X1,
              float* Y, float* Xhalf, float* X_opt, float* gbar_opt, void* stream);
int lq_message_modified(lq_plan* plan);

/* Code-length accounting (appendix on the coding framework).
 * lq_level_probabilities: for every layer, the probability p^_j that level j is emitted,
 *   p^_j = int hat_j(u) dF~(u), with F~ the CDF estimate of lq_fit_levels (the num_samples histograms
 *   merged with the weights N_z^2 / sum N_z^2, linear inside a bin, the last bin a point mass at u = 1) and
 *   hat_j the rounding probabilities towards l_j from its two neighbouring intervals.  The expected number of
 *   non-zero coordinates of the layer is (1 - p^_0) d_m and the appendix's expected length in bits is
 *   32 + (1 - p^_0) d_m + (1 - sum_{j=1}^{n-2} p^_j log2 p^_j) d_m.
 *   hist dev [num_samples][L][LQ_HIST_STRIDE], norms dev [num_samples][L] as for lq_fit_levels;
 *   staged = 0: the levels of the latest lq_quantize_pack, 1: the staged levels (latest set / fit);
 *   probs dev [L][256] doubles out (entries past the layer's level count are 0; a layer without mass gives 0s).
 * lq_symbol_counts: counts[k][m][j] += number of coordinates of layer m in worker k's message that carry
 *   level index j (padding excluded).  packed dev [K][W]; counts dev [K][L][256] u32, caller-zeroed. */
int lq_level_probabilities(const lq_plan* plan, const uint32_t* hist, const float* norms, int32_t num_samples,
                           int32_t staged, double* probs, void* stream);
int lq_symbol_counts(const lq_plan* plan, const uint32_t* packed, uint32_t* counts, void* stream);

/* Entropy stage on top of the fixed-width message (appendix on the coding framework: with the level
 * frequencies known or estimated, a Huffman code on the level symbols; one sign bit per non-zero entry).
 * A layer's code is a list of word lengths, 1..LQ_CODE_MAX_LEN bits, one per level index; the words are the
 * canonical ones (symbols ordered by length, then index; first word all zeros, each next word the previous
 * plus one, shifted left where the length grows), sent most significant bit first.  Every layer starts with
 * the flat code (b bits per index).
 *   lq_code_build   (host only, no device work): Huffman lengths for the weights (probabilities or counts,
 *                   e.g. from lq_level_probabilities / lq_symbol_counts); every symbol gets a word, and words
 *                   longer than LQ_CODE_MAX_LEN are avoided by raising the smallest weights.
 *   lq_code_universal (host only): the word lengths of Elias' recursive code of j + 1 for level index j - the
 *                   appendix's choice when only "smaller values are more frequent" is known, no frequencies: 1, 3,
 *                   3, 6 x 4, 7 x 8, 11 x 16, 12 x 32 bits.  The stage sends the canonical words of these lengths,
 *                   so the stream has the recursive code's size.  LQ_EINVAL when a word would exceed
 *                   LQ_CODE_MAX_LEN (n > 63).
 *   lq_code_set/get: lengths host [n], n = 2^b of the layer; set refuses lengths that violate Kraft's inequality
 *                   and synchronises the device.
 * Stream of one worker: the layout's blocks of 1024 coordinates, layer after layer, each starting on a 32-bit
 * word; inside a block the coordinates in the order s = 32 lane + p (coordinate 128 (p / 4) + 4 lane + p % 4),
 * padding left out; per coordinate the level's word and, for a non-zero index, the sign bit; stream bit t of a
 * block is bit t % 32 of its word t / 32.
 *   lq_entropy_encode: packed dev [K][W] -> stream_words dev [K][capacity_words] and block_offsets dev
 *                   [K][lq_plan_blocks() + 1] (first word of every block; the last entry is the worker's length in
 *                   words).  A worker whose stream does not fit keeps its offsets but loses the blocks that do not fit:
 *                   compare the last offset with capacity_words.  (W words always suffice for the flat code.)
 *                   run_offsets: NULL, or dev [K][lq_plan_blocks()][LQ_CODE_RUNS] u16 that receives, for every block,
 *                   the bit offsets inside the block's stream at which its LQ_CODE_RUNS = 8 runs of 128 coordinates
 *                   (four lanes) start: side data of 16 bytes per block (1/8 bit per coordinate) that is not part of
 *                   the stream and lets the decoder work on the eight runs of a block in parallel.
 *                   The call uses scratch that the plan allocates at the first use of the stage (64 bytes per block
 *                   and worker): two encodes of one plan must not overlap on the GPU.
 *   lq_entropy_decode: the inverse, packed fully overwritten; it equals the encoded message except that the sign
 *                   bit of a coordinate with level index 0 comes back as 0 (the stream carries no sign there; the
 *                   decoded value is zero either way).  With run_offsets (as written by lq_entropy_encode for this
 *                   stream) one thread decodes each run of 128 coordinates, and runs of untouched rows are not
 *                   walked; with NULL one thread walks a whole block (an order of magnitude slower).  A stream with no valid word, a block that runs past its end,
 *                   or a run that does not end where the next one starts, sets a flag that lq_entropy_status
 *                   returns (and clears); nothing faults. */
#define LQ_CODE_MAX_LEN 12
#define LQ_CODE_RUNS    8
int lq_code_build(const double* weights, int32_t n, uint8_t* lengths);
int lq_code_universal(int32_t n, uint8_t* lengths);
int lq_code_set(lq_plan* plan, int32_t layer, const uint8_t* lengths, int32_t n);
int lq_code_get(lq_plan* plan, int32_t layer, uint8_t* lengths, int32_t n);
int64_t lq_plan_blocks(const lq_plan* plan);        /* blocks of 1024 coordinates per worker, all layers */
int lq_entropy_encode(lq_plan* plan, const uint32_t* packed, uint32_t* stream_words, int64_t capacity_words,
                      uint32_t* block_offsets, uint16_t* run_offsets, void* stream);
int lq_entropy_decode(lq_plan* plan, const uint32_t* stream_words, int64_t capacity_words,
                      const uint32_t* block_offsets, const uint16_t* run_offsets, uint32_t* packed, void* stream);
int lq_entropy_status(lq_plan* plan, uint32_t* host_flag);

/* Ergodic average (the guarantees of Section 5 are stated for X-bar_{T+1/2} = sum_{t=1..T} X_{t+1/2} / T).
 * qoda_set_average registers a caller-owned DEVICE array xsum [D_pad] of fp64 (16-byte aligned; NULL = off, the
 * default) and zeroes it on `stream`; qoda_init zeroes it again.  Every following qoda_step first adds its incoming
 * Xhalf - the point X_{t+1/2} at which the workers' dual vectors of this iteration were evaluated - to xsum, in
 * fp64, then overwrites Xhalf as usual; after T steps xsum / T is the average (T = t - 1 from qoda_get_scalars).
 * Costs one more pass over Xhalf and xsum (20 bytes per coordinate) per step. */
int qoda_set_average(lq_plan* plan, double* xsum, void* stream);

/* Alternative adaptive step sizes (Eq. Alt with the running sums of the appendix on the almost-sure
 * boundedness model): with q_hat in (0, 1/4], every following qoda_step uses
 *   eta_{t+1} = fp32((1 + lambda_{t-1} + mu_{t-1})^(-1/2)),  gamma_{t+1} = fp32((1 + lambda_{t-1})^(q_hat - 1/2)),
 *   lambda_t = sum_{s<=t} ||gbar_{s+1/2}||^2,  mu_t = sum_{s<=t} ||X_s - X_{s+1}||^2  (fp64 sums of squares of
 *   fp32 values; both start at 0 in qoda_init, so eta_1 = eta_2 = gamma_1 = gamma_2 = 1),
 * where gbar is the mean of the K decoded messages: lambda is the appendix's form, the squared norm of the
 * AGGREGATE, sum_s ||sum_k V^_{k,s+1/2}||^2 / K^2, which the proofs use.  The display of Eq. (Alt) in the main
 * text sums the K workers' squared norms instead (sum_s sum_k ||V^_{k,s+1/2}||^2 / K^2, larger by up to a
 * factor K); that form is not computed here.
 * X_{t+1} = fma(eta_{t+1}, Y_{t+1}, X_1), X_{t+3/2} = fma(-gamma_{t+1}, gbar, X_{t+1}), and adds this
 * iteration's terms to lambda and mu afterwards.  The statistic of lq_quantize_pack is not used, so
 * its prev_packed / prev_norms may be NULL; while this schedule is on, lq_quantize_pack does not compute it
 * either (lq_get_statistics then reads zeros), except in calls that also collect histograms.  q_hat = 0 switches back to Eq. (general_stepsize).
 * Choose the schedule before qoda_init: the two schedules keep separate sums. */
int qoda_set_alt_rates(lq_plan* plan, double q_hat);
/* Host copies of lambda, mu and the current gamma; synchronises.  Any output may be NULL. */
int qoda_get_alt_scalars(const lq_plan* plan, double* lambda, double* mu, double* gamma);

/* Host copies of the QODA scalars (t = index of the next iteration, S, eta); synchronises.
 * Any output may be NULL. */
int qoda_get_scalars(const lq_plan* plan, int64_t* t, double* S, double* eta);

/* Per-(worker, layer) squared differences left by the last lq_quantize_pack
 * (host_sq_diff [K][L] doubles) and status flags (host_flags [K][L], LQ_STATUS_*) of the
 * last norm computation.  Either may be NULL.  Synchronises. */
int lq_get_statistics(const lq_plan* plan, double* host_sq_diff, uint32_t* host_flags);

/* L^q norm of one device vector with no allocation anywhere (the paper has no counterpart: this is
 * a convenience of the library).  For callers that cannot allocate device memory when they need a
 * norm - all device memory already belongs to another allocator, or the device-wide
 * synchronisation that cudaMalloc and cudaFree imply is not acceptable where the call sits - and
 * who therefore cannot create a plan.  The scratch of the two-stage reduction is a fixed array
 * inside the library image (32 KB on every GPU that loads the library, held until the process
 * exits), so this call and everything below it call no cudaMalloc, cudaFree or allocating routine.
 *   v dev [n] fp32, 16-byte aligned (may be NULL when n = 0);  n in [0, 134217728] (4096 tiles of
 *   32768 values: larger n is refused with LQ_EINVAL);  q as in lq_plan_create (0 = infinity
 *   norm, 1..16);  norm_out dev [1]: fp32(||v||_q) accumulated in fp64, or 0 when flagged;
 *   status_out dev [1] or NULL: 0, LQ_STATUS_ZERO_NORM or LQ_STATUS_NONFINITE.
 * Asynchronous on `stream`.  The first call on each device looks up the array's device address
 * (cudaGetSymbolAddress, which may load the module on that device); make that first call before
 * any stream capture begins.  All calls share the one array and every call overwrites the
 * entries it reads back, so nothing needs clearing, but calls that overlap on the GPU (two
 * streams, two host threads) race on it: order them. */
int lq_vector_norm_static(const float* v, int64_t n, int32_t q, float* norm_out, uint32_t* status_out,
                          void* stream);

/* Measurement aid (no counterpart in the paper).  While enabled, every kernel the library
 * launches for this plan is bracketed by two CUDA events on the caller's stream.
 * lq_profile_read synchronises the device, returns per kernel the summed device time in
 * milliseconds and the number of launches since the last read (arrays of LQ_NUM_KERNELS,
 * indexed by LQ_KERNEL_*), and clears the record.  At most 65536 launches are recorded
 * between two reads. */
#define LQ_KERNEL_NORM_PARTIAL   0
#define LQ_KERNEL_NORM_FINALIZE  1
#define LQ_KERNEL_QUANTIZE_PACK  2
#define LQ_KERNEL_STAT_FINALIZE  3
#define LQ_KERNEL_QODA_SCALARS   4
#define LQ_KERNEL_DECODE         5
#define LQ_KERNEL_FIT            6
#define LQ_KERNEL_ALT_FINALIZE   7
#define LQ_KERNEL_AVERAGE        8
#define LQ_KERNEL_BLOCK_LIVE     9
#define LQ_NUM_KERNELS           10
int lq_profile_enable(lq_plan* plan, int32_t enable);
int lq_profile_read(lq_plan* plan, double* total_ms, int64_t* launches);

const char* lq_error_string(int code);
const char* lq_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* LQ_H_ */
