/*
 * qsparse.h — C boundary of the Qsparse-local-SGD synchronisation round for one B200.
 *
 * The library holds R simulated workers as an R x d fp32 batch in the memory of ONE
 * GPU and runs, with its own sm_100a kernels, one synchronisation step of
 * Qsparse-local-SGD (Basu, Data, Karakus, Diggavi; Algorithm 1, and Algorithm 2 for
 * the asynchronous variant):
 *
 *   worker r :  u_r = m_r + (x - xw_r)            argument of the compressor (Alg. 1, worker branch)
 *               g_r = Q Comp_k(u_r)               composed operator (Section 2.3, Lemmas 1-3;
 *                                                 per-segment by Corollary 1)
 *               m_r <- u_r - g_r                  memory update (Alg. 1, worker branch)
 *               g_r -> wire record                "send g to the master"
 *   master   :  x <- x - (1/R) sum_r g_r          (Alg. 1, master branch; sum over the
 *                                                 participating set S in Alg. 2, divisor still R)
 *               xw_r <- x                         broadcast
 *
 * Conventions common to every call
 *   - All array arguments named "device" are pointers into the memory of the GPU that
 *     was current when qs_init ran; "host" arrays are ordinary host memory and are
 *     read before the call returns.  The caller owns every buffer it passes; the
 *     library owns only its scratch, freed by qs_destroy.
 *   - x is d floats; xw, mem (and anchors) are R x d floats, row r = worker r,
 *     rows contiguous (row stride d).  No alignment beyond 4 bytes is required, but
 *     the 128-bit fast path is taken only when d is a multiple of 4 and the bases are
 *     16-byte aligned.
 *   - Calls enqueue work on the stream given to qs_init and return at once.  The
 *     return value reports argument and launch errors; errors found on the device
 *     (non-finite input, a bounded wait that ran out) are recorded in a device status
 *     word that qs_sync_status reads after synchronising the stream.
 *   - Status codes: QS_OK = 0, negative = error.  Nothing is printed, nothing aborts.
 *   - worker_mask: host array of R bytes, non-zero = worker takes part; NULL = all.
 *   - R <= 32, 1 <= k <= d <= 2^32 - 4096 (coordinates are counted in 32 bits, in tiles of
 *     2048), 1 <= s <= 65535, round < 2^56, R x nseg <= 16384 (up to 2048 (worker, segment)
 *     units their table lives in shared memory; beyond that it is read from global memory).
 *
 * Arithmetic (identical, operation for operation, to the CPU checker under oracle/):
 *   fp32 with no fused multiply-add; u = mem + (x - xw); Top_k orders by the bit
 *   pattern of |u| (larger first), ties by lower index, and always keeps exactly k
 *   coordinates; Rand_k keeps the k smallest (h_i, i) with h_i a Philox4x32-10 word;
 *   norms are the exactly rounded sum of squares (magnitudes), see qs_compress_feedback.
 */
#ifndef QSPARSE_H
#define QSPARSE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct qs_ctx qs_ctx;

enum {
    QS_OK = 0,
    QS_INVALID_ARG = -1, /* bad argument; nothing was enqueued                         */
    QS_ALLOC = -2,       /* scratch allocation failed                                  */
    QS_CUDA = -3,        /* a CUDA runtime call failed; see qs_last_error              */
    QS_CAPACITY = -4,    /* caller's wire stride is smaller than qs_wire_words         */
    QS_NONFINITE = -5,   /* an inf or NaN reached the compressor (device status)       */
    QS_STATE = -6,       /* call out of order (no buffers bound, nothing compressed)   */
    QS_TIMEOUT = -7,     /* a bounded device-side wait ran out (device status)         */
    QS_TOO_LARGE = -8    /* d beyond QS_STATIC_MAX_D (qs_unpack_accumulate_static only) */
};

/* Sparsifiers of Section 2.2. */
#define QS_TOPK 0
#define QS_RANDK 1
/* Quantizers: QSGD s-level stochastic (Definition 1, example 1) composed without scaling
 * (Lemma 1) or divided by 1 + beta_{k,s} (Lemma 2); Sign scaled by the l1 norm over k
 * (Definition 2, Lemma 3 with m = 1). */
#define QS_QSGD 0
#define QS_QSGD_SCALED 1
#define QS_SIGN_L1 2
/* No quantizer: the sparsifier alone (a compression operator with gamma = k/d, Section 2.2; the
 * Top_k-SGD scheme the paper compares with).  g = u on the kept set; the record carries the
 * kept values as 32-bit words in place of the sign and level streams, all k of them. */
#define QS_NONE 3
/* Sign scaled by the l2 norm over k (Lemma 3 with m = 2; gamma_2 = 1/d): g = +-N2/k with N2 the
 * exactly summed l2 norm of the kept vector; record as for QS_SIGN_L1.  m >= 3 is not provided. */
#define QS_SIGN_L2 4
/* Stochastic s-level quantizer between the smallest entry lo and the largest entry hi of the kept
 * vector (Definition 1, example 2): levels lo + j D, j = 0 .. s-1, D = (hi - lo)/(s - 1); an entry
 * goes to the level below or above it, up with probability (v - lo)/D - floor((v - lo)/D)
 * (unbiased).  fp32: p = (v - lo)/D; j = min(floor(p) + (U < p - floor(p)), s - 1) with U the top
 * 24 bits of the Philox word of stream 0; g = lo + j * D (product and sum rounded on their own);
 * hi == lo gives j = 0.  Needs s >= 2.  Every kept entry is sent: in the record the count is
 * implied (n = k_seg), the segment's header pair carries (lo, hi), there is no sign stream and
 * the level stream holds j; bits = 64 + k (b_idx + b_lvl) per segment.  qs_export_selection
 * reports the levels as j + 1 and hi as the norm. */
#define QS_MINMAX 5
/* op argument of qs_init */
#define QS_OP(sparsifier, quantizer) ((sparsifier) | ((quantizer) << 4))

/* Round argument meaning "use the context's counter, then increment it". */
#define QS_ROUND_AUTO UINT64_MAX

/*
 * qs_init — create a context for R workers of d coordinates, keeping k per worker with
 * an s-level quantizer (Section 2; Algorithm 1 line 1 fixes the zero initial state, which
 * is the caller's to provide in the buffers it binds).
 *   out          receives the context (host pointer).
 *   op           QS_OP(sparsifier, quantizer).
 *   seed         key of the Philox4x32-10 generator; the word for (round, worker,
 *                element, stream) uses counter (element >> 2, worker, round_lo,
 *                (round_hi << 8) | stream) and output word element & 3; stream 0 feeds
 *                the quantizer, stream 1 the Rand_k subset.
 *   cuda_stream  a cudaStream_t (NULL = the legacy default stream).
 * Allocates all scratch (candidate storage sized for the worst case, 20 R d bytes, 24 for
 * Rand_k, plus 4 d bytes of sender bits and small tables); one
 * segment [0, d) with k is installed.  Returns QS_INVALID_ARG, QS_ALLOC or QS_CUDA on
 * failure, in which case *out is NULL.
 * Read from the environment here, for tuning and tests (results never depend on them):
 * QSPARSE_UNIT_CAP (0..6144, default 6144: the longest candidate list that one thread
 * block may select from on its own; 0 sends every list through the grid-wide radix
 * levels), QSPARSE_ORDER_EVEN_MAX (0..2048, default 2048: (worker, super-block) pairs up to
 * which the order stage deals candidates evenly; 0 = always by region), QSPARSE_BLOCK_PACK
 * (whole rounds pack the records block by block before the closing stage, not by spare warps
 * beside it), QSPARSE_MID_PER_SM (thread blocks of the persistent kernel per SM, default
 * 4), QSPARSE_NO_TMA (dense pass with plain loads), QSPARSE_TMA_DEPTH (its ring depth),
 * QSPARSE_SPIN_LIMIT (polls a grid barrier waits before it gives up with QS_TIMEOUT; default
 * 2^22, about a second) and QSPARSE_TEST_MISS_BARRIER (test of that path: in the first
 * persistent launch of the context one block stays away from the first barrier, so that every
 * other block's bounded wait runs out).
 */
int qs_init(qs_ctx** out, int R, int64_t d, int64_t k, int s, int op, uint64_t seed,
            void* cuda_stream);

/*
 * qs_set_segments — piecewise operator of Corollary 1: segment g covers coordinates
 * [offsets[g], offsets[g+1]) and keeps k_seg[g] of them with its own norm and scaling.
 *   offsets (host, nseg+1, offsets[0] = 0, increasing, offsets[nseg] = d), k_seg (host,
 *   nseg, 1 <= k_seg[g] <= segment length).  Reallocates the tables; resets the
 *   threshold predictions.  Synchronises the stream.
 */
int qs_set_segments(qs_ctx* ctx, int nseg, const int64_t* offsets, const int64_t* k_seg);

/*
 * qs_bind — give the context the state it works on (all device, caller-owned):
 *   x global model (d), xw local models (R x d), mem memories (R x d),
 *   anchors (R x d) or NULL.  anchors == NULL selects Algorithm 1 (every worker's
 *   reference point is x); with anchors the rounds follow Algorithm 2: worker r forms
 *   its update from anchors_r, and a broadcast also overwrites anchors_r.
 */
int qs_bind(qs_ctx* ctx, float* x, float* xw, float* mem, float* anchors);

/*
 * qs_set_sharding — the masterless form of the method (Section 1: each worker exchanges its
 * updates with all other workers and the aggregation is done without a master), for a job of
 * R_total workers spread over several contexts, one per GPU: this context holds the workers
 * worker_base .. worker_base + R - 1.  After the call
 *   - the random draws (QSGD levels, Rand_k) use the global worker id, so a worker's record does
 *     not depend on where it runs;
 *   - qs_unpack_accumulate expects the records of the whole job: wire rows and worker_mask are
 *     indexed by global worker id (R_total rows), and the update divides by R_total;
 *   - qs_compress_feedback, qs_pack, qs_broadcast, qs_local_step keep local indices (R rows);
 *   - qs_sync_round and qs_sync_round_step return QS_STATE unless R_total == R: the records of
 *     the other shards have to be gathered between qs_pack and qs_unpack_accumulate.
 * Every shard decodes the same R_total records in the same order, so the replicas of x stay
 * bit-identical.  Requires worker_base >= 0 and worker_base + R <= R_total <= 32.
 */
int qs_set_sharding(qs_ctx* ctx, int worker_base, int R_total);

/*
 * qs_local_step — the local SGD step of Algorithm 1 (line 5) for the masked workers:
 *   xw_r <- xw_r - eta * grad_r, a multiply and a subtract, each rounded to fp32.
 *   grad: device, R x d.
 */
int qs_local_step(qs_ctx* ctx, const float* grad, float eta, const uint8_t* worker_mask);

/*
 * qs_local_step_momentum — the local step with momentum on the local iterations, as the
 * experiments of Section 5.1 run it (momentum 0.9; the paper prints no formula, the
 * heavy-ball form is taken), for the masked workers:
 *   vel_r <- mu * vel_r + grad_r ;  xw_r <- xw_r - eta * vel_r
 * every product and sum rounded to fp32 on its own.  grad, vel: device, R x d; vel is
 * caller-owned and updated in place.  mu = 0 gives qs_local_step (and vel_r = grad_r).
 */
int qs_local_step_momentum(qs_ctx* ctx, const float* grad, float* vel, float eta, float mu,
                           const uint8_t* worker_mask);

/*
 * qs_compress_feedback — worker half of a synchronisation (Alg. 1 lines 9-10; Alg. 2
 * lines 9-10) for the masked workers: forms u, finds the kept set of each segment,
 * computes the norm of the kept k-vector (the quantizer acts on it as a length-k
 * vector, proof of Lemma 1), the levels and signs, and writes m <- u - g into mem.
 * The result (indices, levels, signs, norms, counts) stays in scratch for qs_pack.
 *   Norm: the exact sum of the squares (QSGD) or magnitudes (Sign) of the kept values,
 *   rounded once to fp64; sqrt in fp64 for QSGD; rounded to fp32.
 *   Level: a = |u| * s; p = a / N; l = floor(p); U = (w >> 8) * 2^-24;
 *   level = min(l + (U < p - l), s); N == 0 gives level 0.
 *   Value: QSGD g = (N * level) / s (times fl32(1 / (1 + beta_{k,s})) when scaled,
 *   beta_{k,s} = min(k / s^2, sqrt(k) / s)); Sign g = N1 / k; negated when u < 0.
 * Non-finite u sets QS_NONFINITE in the device status.
 */
int qs_compress_feedback(qs_ctx* ctx, uint64_t round, const uint8_t* worker_mask);

/*
 * qs_pack — "send g to the master" (Alg. 1 line 9): writes the records of the last
 * qs_compress_feedback.  wire: device, R rows of stride_words 32-bit words; row r:
 *   directory: nseg pairs (n, norm bits); then for each segment three streams, each
 *   padded to a word, fields LSB first: n segment-local indices (ascending) of
 *   max(1, ceil(log2 d_seg)) bits; n sign bits; for QSGD n fields (level - 1) of
 *   max(1, ceil(log2 s)) bits.  QSGD drops level-0 entries, Sign sends all k.  Words
 *   after the record, up to qs_wire_words, are zero.
 * bits_out: device, R int64, or NULL: exact record size in bits,
 *   sum over segments of 64 + n (b_idx + 1 + b_lvl).
 * Rows of workers outside the last mask are not written.
 * Returns QS_CAPACITY (nothing written) if stride_words < qs_wire_words(ctx).
 */
int qs_pack(qs_ctx* ctx, uint32_t* wire, int64_t stride_words, int64_t* bits_out);

/*
 * qs_unpack_accumulate — master (Alg. 1 line 17; Alg. 2 line 18): decodes the records
 * of the masked workers from the wire words alone and updates x at every index some
 * worker sent: acc = 0; acc += g_r in increasing r; x <- x - acc / R.
 */
int qs_unpack_accumulate(qs_ctx* ctx, const uint32_t* wire, int64_t stride_words,
                         const uint8_t* worker_mask);

/*
 * qs_broadcast — Alg. 1 lines 11 and 18 (Alg. 2 lines 11 and 18): xw_r <- x, and
 * anchors_r <- x when anchors are bound, for the masked workers.
 */
int qs_broadcast(qs_ctx* ctx, const uint8_t* worker_mask);

/*
 * qs_sync_round — the whole synchronisation for the masked workers, with the same final
 * bytes in x, xw, mem, anchors, wire and bits_out as qs_compress_feedback, qs_pack,
 * qs_unpack_accumulate, qs_broadcast in that order, in two kernel launches: the dense pass
 * that forms u, and one persistent kernel that runs every later step and ends with the
 * broadcast.  wire / stride_words / bits_out as in qs_pack.
 */
int qs_sync_round(qs_ctx* ctx, uint64_t round, const uint8_t* worker_mask, uint32_t* wire,
                  int64_t stride_words, int64_t* bits_out);

/*
 * qs_sync_round_step — the local step that precedes a synchronisation (Alg. 1 line 5; Alg. 2
 * line 5) taken inside the round: the same final bytes in x, xw, mem, anchors, vel, wire
 * and bits_out as qs_local_step (vel == NULL) or qs_local_step_momentum (vel != NULL) for
 * the masked workers followed by qs_sync_round with the same mask.  The half-step model
 * xw_r - eta * (...) is formed in the dense pass and never written: the broadcast that
 * ends the round overwrites xw_r anyway, which saves one read and one write of xw_r.
 * grad (and vel): device, R x d; rows of workers outside the mask are neither read nor
 * written.  Rows that are not 16-byte aligned take the two calls named above instead.
 */
int qs_sync_round_step(qs_ctx* ctx, const float* grad, float* vel, float eta, float mu,
                       uint64_t round, const uint8_t* worker_mask, uint32_t* wire,
                       int64_t stride_words, int64_t* bits_out);

/*
 * qs_export_selection — copies the result of the last compression, after it has been packed
 * (qs_pack or qs_sync_round), out of scratch, for
 * checking against a reference (all device, any may be NULL):
 *   sel_idx  R x K int64, global indices of the kept sets, ascending, segments in order
 *            (K = sum of k_seg);  level R x K int32 (Sign: 1);  sign R x K bytes (1 = u < 0);
 *   norm R x nseg floats;  n R x nseg int64 (entries sent).
 */
int qs_export_selection(qs_ctx* ctx, int64_t* sel_idx, int32_t* level, uint8_t* sign,
                        float* norm, int64_t* n);

/* Words one worker's record can need (n = k in every segment); < 0 on a bad context. */
int64_t qs_wire_words(const qs_ctx* ctx);
/* Bit count of a record whose segments send n[g] entries (host array, nseg). */
int64_t qs_record_bits(const qs_ctx* ctx, const int64_t* n);
/* Sum of k_seg. */
int64_t qs_total_k(const qs_ctx* ctx);

/*
 * Gap-coded records.  The paper measures what the workers send in bits (Section 5, the x-axes
 * of its figures) and leaves the coding of the k indices open.  qs_recode_gaps turns the
 * records of qs_pack / qs_sync_round into a second form in which a segment's ascending indices
 * travel as the first index and the gaps i_j - i_(j-1) - 1 in fields of w bits.  For w >= 1 the
 * field value E = 2^w - 1 is an escape: a gap >= E is sent as E and the gap itself follows, in
 * order, among x exceptions of b_idx bits.  w = 0 (no fields) needs every gap to be 0.  The
 * width is the one in 0 .. b_idx that makes (n - 1) w + x(w) b_idx smallest (the smallest such
 * on a tie), so the form is never longer than the plain one by more than its 6 bits of width.
 * qs_decode_gaps turns the rows back, word for word, for qs_unpack_accumulate.  Row of a worker:
 *   directory: nseg entries of five words (n, norm bits, w, first index, x) (the min/max
 *              quantizer keeps (min, max) in the first two, n = k; x is not counted as sent:
 *              it could be recounted from the fields);
 *   per segment: n - 1 gap fields of w bits, LSB first, padded to a word; x exception fields
 *              of b_idx bits, padded to a word; then the streams that follow the indices in
 *              the plain record (signs, levels or values), unchanged.
 * Words after a record, up to qs_gap_words, are zero.
 *   wire / stride_words     device, rows in the format of qs_pack (stride >= qs_wire_words)
 *   packed / packed_stride  device, rows of packed_stride >= qs_gap_words(ctx) words
 *   worker_mask             host, or NULL for all: one byte per worker of this context for
 *                           qs_recode_gaps (the senders' side: the rows of qs_pack), one per
 *                           worker of the job for qs_decode_gaps (the master's side, see
 *                           qs_set_sharding); rows of workers outside it are neither read nor written
 *   bits_out                device, one int64 per worker, or NULL: exact size in bits,
 *                           sum over segments of 64 + 6 + [n >= 1] (b_idx + (n - 1) w + x b_idx) + n (entry bits - b_idx)
 * Both calls are asynchronous on the context's stream, allocate nothing and keep no state; a
 * count above k_seg, a width above b_idx, more exceptions than fields or a first index outside
 * the segment in the input is clipped (the words read and written stay inside the rows).  QS_CAPACITY (nothing written) when
 * a stride is too small.
 */
int64_t qs_gap_words(const qs_ctx* ctx);
int qs_recode_gaps(qs_ctx* ctx, const uint32_t* wire, int64_t stride_words, const uint8_t* worker_mask,
                   uint32_t* packed, int64_t packed_stride, int64_t* bits_out);
int qs_decode_gaps(qs_ctx* ctx, const uint32_t* packed, int64_t packed_stride, const uint8_t* worker_mask,
                   uint32_t* wire, int64_t stride_words);

/* Synchronises the stream and returns the first error recorded on the device since the
 * last call (QS_OK if none), clearing it.  After a device-side error (QS_NONFINITE,
 * QS_TIMEOUT, QS_STATE) the round that hit it is void: its outputs are undefined, and this call
 * also puts the library's scratch back into its starting state, so call it before the next
 * round. */
int qs_sync_status(qs_ctx* ctx);
/* Text of the last host-side error of this context (never NULL). */
const char* qs_last_error(const qs_ctx* ctx);

/* Round counter used by QS_ROUND_AUTO; with the seed and the bound buffers it is the
 * whole state needed to resume a run. */
uint64_t qs_get_round(const qs_ctx* ctx);
int qs_set_round(qs_ctx* ctx, uint64_t round);

/*
 * qs_get_stats — host counters since qs_init (synchronises the stream): out[0] rounds
 * compressed, out[1] worker-rounds whose predicted threshold missed and took the exact
 * histogram pass, out[2] candidates examined, out[3] kernels launched, out[4] blocks of the
 * persistent kernel (all resident at once).  Writes min(n, 5) values.
 */
int qs_get_stats(qs_ctx* ctx, int64_t* out, int n);

/*
 * qs_enable_phase_timing / qs_get_phase_timing — measurement aid, not part of the method:
 * when on, qs_sync_round records CUDA events on the context's stream around its dense pass.
 * qs_get_phase_timing synchronises and returns, summed over the rounds since the last call
 * and then cleared: ms[0] the dense pass (form u, candidate flags and runs: one kernel launch
 * per round), ms[1] the rest of the round (selection, quantizer, memory update, pack, master
 * update and broadcast: one persistent kernel), ms[2] the number of rounds.  Writes
 * min(n, 3) values.
 */
int qs_enable_phase_timing(qs_ctx* ctx, int on);
int qs_get_phase_timing(qs_ctx* ctx, double* ms, int n);

/*
 * qs_get_stage_trace — measurement aid: microseconds, from the start of the last persistent
 * kernel of this context, at which each of its grid barriers completed (us[1], us[2], ...,
 * -1 = not reached), block 0 left the kernel (us[30]) and the last block did (us[31]);
 * us[0] = 0.  Synchronises the stream.  Writes min(n, 32) values.
 */
int qs_get_stage_trace(qs_ctx* ctx, double* us, int n);

/*
 * qs_unpack_accumulate_static — the master update of qs_unpack_accumulate for callers that
 * must not allocate.  (The paper has no counterpart: this entry point exists for deployment,
 * not for the method.)
 *
 * Who needs it: code that cannot call cudaMalloc when the update has to run — a serving or
 * training loop in which an allocation would synchronise the whole device, a process whose
 * device memory is owned and handed out by another component, a job whose memory budget is
 * already spent.  qs_init allocates, so this call takes no context: the operator is described
 * by plain arguments, and the one piece of scratch the decode needs (a word per coordinate
 * recording which workers sent it) lives in a fixed array inside the library image.  Every GPU
 * that loads the library therefore holds QS_STATIC_MAX_D words (4 MiB) until the process ends.
 *
 *   R, d, k, s, quantizer   as in qs_init, one segment [0, d); d <= QS_STATIC_MAX_D, else
 *                           QS_TOO_LARGE is returned and nothing is enqueued.  QS_NONE (the
 *                           sparsifier alone, 32-bit values in the record) is not decoded
 *                           by this call: QS_INVALID_ARG.
 *   x (device, d)           updated in place: acc = 0; acc += g_r in increasing r;
 *                           x <- x - acc / R, at every index some masked worker sent.
 *   wire (device), stride_words, worker_mask (host, R bytes or NULL)
 *                           records in the format of qs_pack; QS_CAPACITY if stride_words is
 *                           below the size of a full record.  A record whose count exceeds k,
 *                           or an index >= d, is skipped, never followed.
 *   cuda_stream             the work (one memset, two kernels) is enqueued there.
 * It calls no allocator.  The first call on each device looks up the array's device address
 * (cudaGetSymbolAddress, with that device current): make that first call outside any stream
 * capture.  The array is shared by all calls on a device and keeps the last call's contents;
 * each call clears the d words it uses before use, and calls that overlap in time on one GPU
 * (two streams, two threads) race on it — issue them one after another.
 */
#define QS_STATIC_MAX_D (1 << 20)
int qs_unpack_accumulate_static(int R, int64_t d, int64_t k, int s, int quantizer, float* x,
                                const uint32_t* wire, int64_t stride_words,
                                const uint8_t* worker_mask, void* cuda_stream);

/* Frees the scratch and the context (NULL is allowed). */
void qs_destroy(qs_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* QSPARSE_H */
