/*
 * combo_b200 -- one synchronization round of segmented gossip aggregation
 * ("Decentralized Federated Learning: A Segmented Gossip Approach") for N
 * simulated workers whose flat parameter vectors sit in one GPU's memory.
 *
 * C ABI of libcombo_b200.so (CUDA, sm_100a only; there is no CPU or other
 * fallback).  Plain pointers and sizes; the caller owns every buffer.  Unless
 * a function says otherwise, pointers are DEVICE pointers of the current
 * device, calls only enqueue work on the given stream and never synchronise,
 * and the library allocates nothing.
 *
 * Library-owned device memory: a 4-byte status word (combo_device_status) and
 * a ring of 256 tile dispensers, 16 bytes each.  Every launch of the staged
 * aggregation kernel with persistent CTAs takes the next dispenser (its CTAs
 * draw their tiles from it and the last one to leave clears it): ordinary
 * launches cycle through one half of the ring, launches that are being
 * captured into a CUDA graph through the other half.  Ordinary launches in
 * flight at the same time therefore hold different dispensers as long as
 * fewer than 128 staged launches separate them, and a graph replay never
 * shares one with ordinary launches running beside it.  A graph keeps the
 * dispensers it was captured with: two replays (of one graph or of different
 * ones) whose staged kernels could run at the same time must not hold the
 * same dispenser -- do not run a graph concurrently with itself, nor with a
 * graph captured a multiple of 128 staged launches before or after it.
 * Sharing a dispenser loses or repeats tiles (wrong output, no fault).
 *
 * Notation follows the paper: n = N workers, S segments, R model replicas,
 * |D_j| dataset size of worker j, P_l the set of workers providing segment l.
 *
 * Layouts
 *   parameters  [N][P] row-major, worker-major, dense (row pitch = P elements)
 *   idx         int32 [N][S][R]; idx[w][l][r] = r-th peer of worker w for
 *               segment l; each (w,l) row ascending, all entries != w, distinct
 *   weights     float [N], |D_j| > 0, un-normalised; NULL = all equal
 *
 * Segments (Eq. 1; Section 5.1 cuts the model into S equal parts): segment
 * length L = ceil(P/S); segment l covers columns [min(l*L,P), min((l+1)*L,P)),
 * so the last segment is shorter when S does not divide P and trailing
 * segments may be empty.
 */
#ifndef COMBO_B200_H
#define COMBO_B200_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int combo_status;

enum {
    COMBO_OK = 0,                 /* work enqueued (or, for host calls, done)    */
    COMBO_ERR_INVALID_ARG = 1,    /* size out of range, NULL or misaligned pointer */
    COMBO_ERR_ALIAS = 2,          /* input and output ranges overlap             */
    COMBO_ERR_UNSUPPORTED = 3,    /* current device is not compute capability 10.x */
    COMBO_ERR_CUDA = 4,           /* a CUDA runtime call failed; see combo_last_cuda_error */
    COMBO_ERR_DEVICE_TIMEOUT = 5, /* a bounded wait inside a kernel ran out      */
    COMBO_ERR_TOO_LARGE = 6       /* beyond the fixed limit of a no-allocation entry point */
};

/* Limits of this library version. */
#define COMBO_MAX_WORKERS 8192    /* N */
#define COMBO_MAX_SEGMENTS 65536  /* S */
#define COMBO_NOALLOC_MAX_WORKERS 128   /* N of combo_aggregation_divergence_noalloc */

/*
 * Peer selection -- Section 4.1, step (2) "Segments Pulling": every worker
 * issues S*R pull requests; each target is drawn at random from all the OTHER
 * workers, without replacement, until no option is left.  When the pool of
 * N-1 others is exhausted a freshly shuffled pool is opened; peers already
 * chosen for the segment being filled are skipped (P_l of Eq. 3 is a set).
 * Hence: never the worker itself, R distinct peers per (worker, segment), all
 * S*R peers of a worker distinct when S*R <= N-1, otherwise every other worker
 * is used floor or ceil of S*R/(N-1) times.
 *
 * The table is a pure function of (seed, round, N, S, R): random numbers come
 * from a counter-based generator (splitmix64 steps chained over the words
 * seed, round|worker, epoch|position; Fisher-Yates shuffle with the
 * multiply-shift range reduction), so the call can be issued ahead of the
 * local update, as the paper notes for the pull requests.
 *
 * idx_out: device int32[N*S*R], written completely; not touched when R == 0.
 * Requires 1 <= N <= COMBO_MAX_WORKERS, 1 <= S <= COMBO_MAX_SEGMENTS,
 * 0 <= R <= N-1.  combo_select_peers enqueues on the legacy default stream;
 * the _async form on `stream` (a cudaStream_t passed as void*).
 */
combo_status combo_select_peers(uint64_t seed, uint32_t round, int N, int S, int R,
                                int32_t* idx_out);
combo_status combo_select_peers_async(uint64_t seed, uint32_t round, int N, int S, int R,
                                      int32_t* idx_out, void* stream);

/*
 * Segment-wise aggregation -- Eq. 3 and Eq. 4 (Section 3, "Segmented
 * Aggregation"), for all N workers at once:
 *
 *   out[w][p] = sum_{j in P_l(w)} |D_j| * in[j][p]  /  sum_{j in P_l(w)} |D_j|
 *
 * with l the segment that holds column p and P_l(w) = {w} U idx[w][l][0..R).
 * Every worker reads the same pre-aggregation inputs (workers send the model
 * they hold after the local update, Section 4.1 steps 3 and 4), so params_out
 * must not overlap params_in.
 *
 * Arithmetic: binary32, Eq. 3 as it is written.  num = |D_w|*x_w, then
 * num = fma(|D_k|, x_k, num) for the peers in ascending order;
 * den = |D_w| + |D_k1| + ... in the same order; out = num * (1/den), the
 * reciprocal rounded to binary32 (one IEEE division per worker and segment).
 * A single provider is taken as it is (out = x).  With weights == NULL every
 * |D_j| is 1: the products are exact and num is the plain sum in that order
 * (bfloat16 rows are then added by the mixed-precision instruction
 * add.rn.f32.bf16, which widens exactly and rounds once: the same bits).
 * |D_j|*x must stay within the binary32 range.  No fast-math, denormals kept.
 *
 * params_in, params_out: float [N][P], base addresses 16-byte aligned.
 * weights: float[N] or NULL.  idx: int32[N][S][R], trusted (see
 * combo_validate_idx); may be NULL when R == 0.  1 <= P, 0 <= R <= N-1.
 * R == 0 copies the input bit for bit.
 */
combo_status combo_segment_aggregate(const float* params_in, float* params_out,
                                     const float* weights, const int32_t* idx,
                                     int N, int64_t P, int S, int R, void* stream);

/*
 * The same with parameters stored as bfloat16 (uint16_t bit patterns):
 * inputs are widened exactly, accumulation is binary32 as above, the result
 * is rounded to nearest even.  Rows need not be 16-byte aligned (odd P*2
 * pitches are handled); the base addresses must be.
 */
combo_status combo_segment_aggregate_bf16(const uint16_t* params_in, uint16_t* params_out,
                                          const float* weights, const int32_t* idx,
                                          int N, int64_t P, int S, int R, void* stream);

/*
 * Local step fused in front of the aggregation -- Section 4.1 step (1) with
 * one SGD step (tau = 1) on a supplied gradient: every worker j first forms
 * x'_j = fma(-lr, grads[j], params_in[j]) (binary32), and Eq. 3 is evaluated
 * on the x'.  Peers contribute their UPDATED rows, exactly as if the step had
 * been applied to all of params_in before combo_segment_aggregate.  grads:
 * float [N][P], 16-byte aligned, must not overlap params_out.
 */
combo_status combo_segment_aggregate_sgd(const float* params_in, const float* grads, float lr,
                                         float* params_out, const float* weights,
                                         const int32_t* idx, int N, int64_t P, int S, int R,
                                         void* stream);

/*
 * Column-sharded form of the three calls above, for a vector of P_total
 * parameters whose columns [p_begin, p_begin + width) are held locally as
 * [N][pitch] arrays (pitch >= width elements; local column 0 = global column
 * p_begin).  Eq. 3 couples workers only at equal p, so shards need no
 * exchange; segment bounds are those of the P_total-vector.
 * elem_bytes: 4 = float, 2 = bfloat16.  grads may be NULL (no local step;
 * must be NULL for bfloat16).
 */
combo_status combo_segment_aggregate_cols(const void* params_in, const void* grads, float lr,
                                          void* params_out, int elem_bytes,
                                          const float* weights, const int32_t* idx,
                                          int N, int64_t P_total, int S, int R,
                                          int64_t p_begin, int64_t width, int64_t pitch,
                                          void* stream);

/*
 * Worker-sharded form -- Section 3 "Segmented Pulling" (Eq. 2) followed by
 * Eq. 3, for workers spread over several GPUs of one node.  d_rows: DEVICE
 * array of N pointers, d_rows[j] = flat model of worker j (P elements, 16-byte
 * aligned), in this GPU's memory or in a peer GPU's memory that is mapped
 * into this process (peer access / symmetric memory).  The call forms the new
 * models of the n_local workers w_begin .. w_begin + n_local - 1 that this
 * GPU hosts and writes them to out, [n_local][out_pitch] (out_pitch >= P
 * elements, out_pitch * elem_bytes a multiple of 16; must not overlap any
 * row).  A pull is a plain load of W_k[l] from where worker k lives (no bulk
 * copy, no multicast); a segment of a peer that several hosted workers pull
 * is loaded once per column tile and shared, so per segment index at most R
 * segments per hosted worker cross to this GPU -- the paper's count, less the
 * shared ones.  idx is the full [N][S][R] table (every GPU computes the same
 * one from the seed), weights the full [N] array or NULL.  Same arithmetic and
 * order as combo_segment_aggregate.  The caller orders the rounds: rows must
 * be final before the call (Section 4.1: a worker sends after its local
 * update) and must not be overwritten while any GPU still reads them.
 */
combo_status combo_segment_aggregate_rows(const void* const* d_rows, void* out, int64_t out_pitch,
                                          int elem_bytes, const float* weights, const int32_t* idx,
                                          int N, int64_t P, int S, int R, int w_begin, int n_local,
                                          void* stream);

/* Debug helper for the call above: *dev_flag (device int32) becomes 0 when all
 * N row pointers are non-null and 16-byte aligned, else 1 + the first bad row. */
combo_status combo_check_rows(const void* const* d_rows, int N, void* stream, int32_t* dev_flag);

/*
 * Dynamic workers -- Section 4.2.
 *
 * combo_select_peers_online: a worker that is offline is not pulled from (its
 * requester turns to some other worker instead), so every online worker
 * draws its peers from the ONLINE others only, by the same procedure as
 * combo_select_peers (identical tables when all are online).  An offline worker
 * issues no requests: its rows are filled with -1.  h_online: HOST array of N
 * bytes, non-zero = online (membership is decided on the host); NULL = all
 * online.  Requires R <= (online workers) - 1.
 *
 * combo_segment_aggregate_members: Eq. 3 with the provider set
 *   P_l(w) = ({w} unless w is a newcomer) U { idx[w][l][r] : idx[w][l][r] >= 0 }.
 * A newcomer has no model of its own yet: it aggregates the segments it
 * pulled without an own term (Section 4.2), so its row is never read; a
 * negative idx entry is a pull that found no online peer.  A worker left with no provider (an offline
 * worker's -1 rows) keeps its own values.  h_newcomer: HOST array of N bytes,
 * non-zero = newcomer, or NULL.  Same arithmetic and order as
 * combo_segment_aggregate (providers in the order self, peers ascending); all
 * entry points above accept negative idx entries in the same way (the
 * worker-sharded call too; it has no newcomer flags).  Rows that are read must
 * hold finite values.
 */
combo_status combo_select_peers_online(uint64_t seed, uint32_t round, int N, int S, int R,
                                       const uint8_t* h_online, int32_t* idx_out, void* stream);
combo_status combo_segment_aggregate_members(const void* params_in, void* params_out, int elem_bytes,
                                             const float* weights, const int32_t* idx,
                                             const uint8_t* h_newcomer, int N, int64_t P, int S, int R,
                                             void* stream);

/*
 * Checks an idx table on the device: every entry in [0,N), != its worker,
 * each (w,l) row strictly ascending.  dev_flag: device int32, set to 0 first,
 * then to 1 + (index of an offending entry) if any check fails.
 */
combo_status combo_validate_idx(const int32_t* idx, int N, int S, int R, void* stream,
                                int32_t* dev_flag);

/*
 * Whole rounds from HOST memory (the paper's worker iteration, steps 2-4, for
 * all workers): copies h_params_in (and h_grads, h_weights when given) to the
 * device buffers, then for t = round .. round+rounds-1 selects peers for
 * (seed, t) and aggregates, ping-ponging between d_in and d_out, and copies
 * the final parameters to h_params_out; all on `stream`, which is
 * synchronised before returning.  With h_grads the fused local step uses the
 * same gradient array in every round.  Host buffers should be page-locked
 * for full copy speed.  Device buffers are the caller's: d_in, d_out (and
 * d_grads if h_grads != NULL) [N][P] of elem_bytes each, d_weights float[N]
 * (if h_weights != NULL), d_idx int32[N*S*R].  h_idx_out, if not NULL,
 * receives the peer table of the last round.  rounds >= 1.
 * Columns are independent in Eq. 3, so the call cuts the vector into column
 * chunks and overlaps the copy-in of one chunk, all rounds of the previous
 * one and the copy-out of the one before on three streams (two of them, and
 * a few events, are created by the first call on a device and kept).  Not
 * reentrant per device.  After the call d_in and d_out hold intermediate
 * rounds, not a defined result.
 */
combo_status combo_round_host(const void* h_params_in, const void* h_grads, float lr,
                              void* h_params_out, int elem_bytes, const float* h_weights,
                              uint64_t seed, uint32_t round, int rounds, int N, int64_t P, int S,
                              int R, void* d_in, void* d_grads, void* d_out, float* d_weights,
                              int32_t* d_idx, int32_t* h_idx_out, void* stream);

/*
 * Aggregation divergence -- Section 4.3, Definition 2 (Eq. 7): for every
 * worker i, rho_i = || W_{t,i} - W_t || (Euclidean norm), where W_{t,i} is row
 * i of `models` (the worker's aggregation result) and W_t is the aggregation
 * of ALL workers, the FedAvg result sum_j |D_j| W_j / sum_j |D_j|, taken over
 * the rows of `mean_of` (the models the round started from).  mean_of == NULL
 * or == models measures the models against their own weighted mean.  With
 * R = N-1 every rho_i is zero up to rounding, as the paper states.
 *
 * models, mean_of: [N][P] dense, elem_bytes 4 (float) or 2 (bfloat16), read
 * only.  rho_out: device double[N].  scratch: device memory of at least
 * combo_divergence_scratch_bytes(N) bytes, 8-byte aligned, used for per-CTA
 * partial sums (no need to clear it; contents are undefined afterwards).
 * Arithmetic: column means and deviations in binary32 (weights normalised
 * first, rows in ascending order), squares summed in binary64; relative error
 * of rho about 1e-6 for models that differ by more than 1e-3 of their size.
 * Two launches on `stream`, no synchronisation.
 */
size_t combo_divergence_scratch_bytes(int N);
combo_status combo_aggregation_divergence(const void* models, const void* mean_of, int elem_bytes,
                                          const float* weights, int N, int64_t P, double* rho_out,
                                          void* scratch, size_t scratch_bytes, void* stream);

/*
 * combo_aggregation_divergence for callers that cannot allocate device memory.
 * (The paper has no counterpart: this is a packaging variant of the call above,
 * same arithmetic, same result.)
 *
 * Who needs it: code that runs where cudaMalloc is not an option -- inside a
 * region being captured into a CUDA graph or between other work that must not
 * synchronise the device (cudaMalloc and cudaFree may do both), in a process
 * whose memory pool is owned and fully handed out by another component, or
 * in a host language binding that cannot create device buffers at all.  Such
 * a caller still passes its inputs and the output, but no scratch: the
 * partial sums go to a fixed array inside the library, 1 MiB that every GPU
 * loading the library holds until the process exits.
 *
 * Limits and rules:
 *  - N <= COMBO_NOALLOC_MAX_WORKERS (128); more returns COMBO_ERR_TOO_LARGE
 *    and combo_last_cuda_error() says so.  P is not limited.
 *  - The first call on each device looks the array's device address up
 *    (cudaGetSymbolAddress, with that device current) and keeps it; make that
 *    first call outside any stream capture.  No call allocates or frees.
 *  - All calls on a device share the one array and it keeps whatever the last
 *    call left.  Nothing has to be cleared, because every partial sum is
 *    written before it is read; but two calls that overlap on the GPU (other
 *    streams, other host threads) race on it -- serialise them on one stream.
 */
combo_status combo_aggregation_divergence_noalloc(const void* models, const void* mean_of,
                                                  int elem_bytes, const float* weights, int N,
                                                  int64_t P, double* rho_out, void* stream);

/*
 * Reads and clears the device status word that kernels set when one of their
 * bounded waits gives up.  Synchronises the device.  Returns COMBO_OK or
 * COMBO_ERR_DEVICE_TIMEOUT (or COMBO_ERR_CUDA).
 */
combo_status combo_device_status(void);

/* Which aggregation kernel the last combo_segment_aggregate* call on this
 * thread launched: 0 none, 1 direct gather, 2 shared-memory staged (persistent
 * CTAs, a ring of tiles), 3 row pull, 5 shared-memory staged with one tile per
 * CTA (short inputs). */
int combo_last_kernel_path(void);

/* Forces a path for the following calls on this thread: 0 automatic (default),
 * 1 direct gather (blocks taken worker-fastest, so that the gather's re-reads
 * are served by L2), 2 staged with persistent CTAs (falls back to direct where
 * staging cannot apply), 5 staged with one tile per CTA (falls back to 2 where
 * rows differ in their 16-byte phase or a tile does not fit), 6 direct gather
 * in the naive order, row after row (the contrast case for profiling: its
 * re-reads mostly come from DRAM); with combo_segment_aggregate_rows: 3 nothing
 * staged. */
void combo_set_kernel_path(int path);

/* Expert knob for the staged kernel, this thread only: tile width in elements
 * (a multiple of 256 up to 2048; for rows whose byte pitch is not a multiple
 * of 16 every 256 asked for become 256 - 16/elem_bytes) and number of pipeline
 * stages; 0 = chosen automatically.  A tile that cannot be honoured makes
 * the call fall back to the direct kernel.  combo_segment_aggregate_rows takes
 * the widest 256 * 2^k columns that do not exceed the tile asked for, and at
 * least three stages. */
void combo_set_tuning(int tile_elems, int stages);

/* This thread only: whether the staged aggregation kernel is launched with
 * programmatic stream serialization (default 1).  With it the kernel may be
 * scheduled while the preceding kernel of the same stream is still draining;
 * it waits for that kernel to complete before its first access to global
 * memory, so stream order as seen through memory is unchanged.  What it
 * hides is launch latency and set-up between back-to-back rounds (Section
 * 4.1: one synchronization per iteration).  0 = ordinary launches. */
void combo_set_launch_overlap(int on);

/* Widest column range a single aggregation launch takes (the staged kernels
 * address columns with signed 32-bit copy coordinates).  Wider inputs are cut
 * into column shards of this many columns inside the call, one launch each;
 * Eq. 3 couples workers only at equal column, so the result is the same. */
int64_t combo_max_launch_columns(void);

/* Expert / test knob, this thread only: cut inputs into shards of `columns`
 * columns instead (rounded down to a multiple of 64; 0 or out of range
 * restores combo_max_launch_columns()). */
void combo_set_launch_columns(int64_t columns);

/*
 * Self-check of the time-out path (no counterpart in the paper).  Every wait
 * inside the kernels is bounded; a wait that runs out sets the device status
 * word and the kernel returns, which combo_device_status() then reports as
 * COMBO_ERR_DEVICE_TIMEOUT.  This call enqueues a one-warp kernel that waits,
 * with a cap of a thousand polls, on a barrier of its own that nothing ever
 * signals, and reports in the same way: after it, combo_device_status()
 * returns COMBO_ERR_DEVICE_TIMEOUT once (site 99 in combo_last_cuda_error())
 * and COMBO_OK afterwards.  It touches no product kernel and leaves nothing
 * armed; the device and the context stay usable.
 */
combo_status combo_debug_dead_wait(void* stream);

const char* combo_status_string(combo_status status);
const char* combo_last_cuda_error(void);
int combo_version(void);

#ifdef __cplusplus
}
#endif
#endif /* COMBO_B200_H */
