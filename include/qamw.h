/*
 * qamw.h -- C ABI of the QAM-W weight codec for NVIDIA B200 (sm_100a).
 *
 * The codec quantises a weight matrix W[d_out, d_in] row by row (paper, Section 3):
 *   encode:  x = W D_s (Section B.2)  ->  r = |x|_2, u = x / r (Section 3.1 step 1)
 *            ->  y = F S u, sign-masked block-Hadamard rotation (step 2, Lemma 1)
 *            ->  pairs z_k = (y_2k, y_2k+1) / sigma_k (steps 3-4, Section 3.4)
 *            ->  idx_k = nearest entry of one 2-D codebook (step 5, Section 3.6)
 *            ->  B = log2 K bits per pair, bit-packed (step 6)
 *   decode:  unpack -> codeword -> x sigma_k -> S F -> x r -> / s_j -> bf16 (Section 3.2, B.2)
 *
 * General rules
 *   - Every function returns QAMW_OK (0) or a negative QAMW_ERR_* code; nothing throws, aborts,
 *     prints or traps.  Argument errors are detected on the host before anything is launched.
 *   - "device" pointers are CUDA global-memory addresses on the current device, "host" pointers
 *     are ordinary process memory.  The caller owns every buffer; the library allocates device
 *     memory only inside a qamw_codebook (released by qamw_codebook_destroy).
 *   - Device-side functions are asynchronous: they enqueue kernels on `stream` (a cudaStream_t
 *     passed as void*, NULL = the default stream) and return without synchronising.
 *   - Matrices are row-major.  W is f32 or bf16 (QAMW_DTYPE_*), with `w_row_stride` elements
 *     between rows; every row must start on a 16-byte boundary.
 *   - Packed rows start `packed_row_stride` bytes apart (>= qamw_packed_row_bytes, a multiple
 *     of 4); index k of a row occupies stream bits [k*B, (k+1)*B), stream bit t being bit
 *     (t mod 8) of byte floor(t/8); padding bits up to the row stride are written as zero.
 *   - Arithmetic contract of the encoder (what makes indices reproducible bit for bit):
 *       t_j = f32(s_j) * sign_j;  x_j = f32(f32(W_ij) * t_j);
 *       r_i = f32(sqrt(sum_j (double)x_j^2));
 *       h   = f32 butterfly of x per block, stages 1, 2, 4, ..., b/2, (a, b) -> (a+b, a-b);
 *       y_j = f32(h_j * g),  g = f32(c_b / r_i) (one f32 division),  c_b = f32(1 / sqrt((double)b));
 *       z   = f32(y * q_k),  q_k = f32(1 / (double)sigma_k);
 *       idx = argmin_c f32(f32(dx*dx) + f32(dy*dy)) with dx = f32(z_x - c_x), dy = f32(z_y - c_y),
 *             lowest index among equal distances.
 *     A row with r_i == 0 is encoded as the origin's codeword in every pair and decodes to zeros.
 *     A row whose norm is not finite sets bit 0 of *status_out; its indices are unspecified.
 */
#ifndef QAMW_H_
#define QAMW_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define QAMW_OK 0
#define QAMW_ERR_ARG (-1)       /* NULL pointer, value out of range */
#define QAMW_ERR_SHAPE (-2)     /* d_in odd or above 16384, block does not divide d_in, K / block not a power of two */
#define QAMW_ERR_ALIGN (-3)     /* pointer or stride alignment */
#define QAMW_ERR_CUDA (-4)      /* a CUDA runtime call failed */
#define QAMW_ERR_NONFINITE (-5) /* reported by qamw_status_to_error for a non-finite row norm */
#define QAMW_ERR_NOMEM (-6)     /* workspace too small / shared memory budget exceeded */

#define QAMW_DTYPE_F32 0
#define QAMW_DTYPE_BF16 1

#define QAMW_FLAG_BRUTE_FORCE 1u /* encode: exhaustive search over all K instead of the cell table */
#define QAMW_FLAG_HALF_DEVICE 2u /* encode, decode, rotate, calibrate: half as many blocks, so that two calls issued on
                                    different streams run side by side and each one's start-up (tables and
                                    per-column constants into shared memory and registers) hides behind the other */

#define QAMW_FLAG_GENERAL_KERNELS 4u /* encode, decode: always run the general row kernels (any d_in, any alignment, any
                                       block size), also where the faster kernels for the common layouts would apply;
                                       same results, meant for testing */

#define QAMW_DEFAULT_SIGN_SEED 0x51A5C0DEC0FFEE01ULL
#define QAMW_MAX_BLOCK 1024 /* cap of Section 3.3 */
#define QAMW_MAX_K 4096
#define QAMW_CALIB_MAX_ROWS 1024 /* row cap of the sigma calibration (Section 3.4) */
#define QAMW_STATIC_SCRATCH_BYTES (16u << 20) /* built-in scratch of qamw_calibrate_static */

typedef struct {
    int32_t d_out, d_in;       /* d_in even, block | d_in, d_in <= 16384 (a row is held by one thread block) */
    int32_t block;             /* b = 2^q, 2 <= b <= 1024 */
    int32_t K;                 /* codebook size, power of two, 2 <= K <= 4096 */
    int32_t w_dtype;           /* QAMW_DTYPE_* of W */
    uint32_t flags;            /* QAMW_FLAG_* */
    int64_t w_row_stride;      /* elements between rows of W (>= d_in) */
    int64_t packed_row_stride; /* bytes between packed rows */
} qamw_params;

typedef struct qamw_codebook qamw_codebook; /* opaque: device copy of C plus its exact search table */

/* ----------------------------------------------------------------------------------------------
 * Host-side helpers (host pointers only, no CUDA calls).
 * -------------------------------------------------------------------------------------------- */

/* Section 3.6: the codebook is the Lloyd-Max quantiser of the unit circular Gaussian.  Sample-based Lloyd
 * on n_samples Box-Muller samples of counter stream `seed` (u = ((mix64(mix64(seed ^
 * 0xD1B54A32D192ED03) + golden*(n+1)) >> 11) + 0.5) * 2^-53, sample i from counters 2i, 2i+1);
 * initial codewords sqrt(2) * sample_i; each iteration assigns every sample to its nearest
 * codeword and moves each codeword to the mean of its cell (empty cells stay); stops when the
 * training MSE improves by no more than rel_tol (relative) or after max_iters updates; the result
 * is sorted by (squared radius, angle) and rounded to f32.
 * codebook_out: host, K*2 floats (x, y interleaved).  train_mse_out: host, may be NULL; receives
 * the mean squared distance of the samples to the returned f32 codebook. */
int qamw_train_codebook(int K, uint64_t n_samples, uint64_t seed, int max_iters, double rel_tol,
                        float* codebook_out, double* train_mse_out);

/* The same training on the current CUDA device (Section 3.6; the paper's Limitations section puts
 * its own trainer at about 5 s per bitrate level and names per-checkpoint codebooks as follow-up).
 * Same rules as qamw_train_codebook: same initial codewords, exact assignment in double (every
 * sample against every codeword, d = dx*dx + dy*dy with one rounding per operation, lowest index on
 * ties), every cell's samples added in sample order, same stopping rule, same final order and f32
 * rounding; the result does not vary from run to run.
 * samples_dev: device, n_samples (x, y) pairs of doubles to train on -- e.g. normalised pairs of a
 * checkpoint -- or NULL: the unit circular Gaussian samples of counter stream `seed` are generated on
 * the device (the device's log / sin / cos may differ from the host's in the last bit).
 * codebook_out: host, K*2 floats.  Optional host outputs (NULL to skip): train_mse_out as in
 * qamw_train_codebook; iters_out: centroid updates done; mse_trace_out: max_iters + 1 doubles, the
 * mean squared distance before every update; seconds_out: wall time of the call.
 * Synchronous; allocates and frees its device scratch (about 32 bytes per sample) itself.
 * n_samples < 2^31. */
int qamw_train_codebook_gpu(int K, uint64_t n_samples, uint64_t seed, const double* samples_dev, int max_iters,
                            double rel_tol, float* codebook_out, double* train_mse_out, int* iters_out,
                            double* mse_trace_out, double* seconds_out);

/* Section B.2: s_j = clamp(r_j^alpha / geomean(r^alpha), 1/16, 16); r_j floored at FLT_MIN;
 * alpha == 0 gives all ones.  act_rms, s_out: host, d_in floats. */
int qamw_channel_scales(const float* act_rms, int d_in, float alpha, float* s_out);

/* Sign mask of Appendix A.1 (a fixed sequence derived from one 64-bit seed):
 * sign_j = -1 if the top bit of mix64(seed + 0x9E3779B97F4A7C15*(j+1)) is set, else +1, with
 * mix64 the SplitMix64 finaliser.  signs_out: host, d_in bytes of +1 / -1. */
int qamw_make_signs(uint64_t seed, int d_in, int8_t* signs_out);

/* Section 3.3: largest power of two dividing d_in, capped at 1024 (2048 -> 1024, 5632 -> 512).
 * Returns 0 for d_in <= 0. */
int qamw_block_size_rule(int d_in);

/* Section 3.1 step 6: ceil((d_in/2) * log2(K) / 8); 0 on invalid arguments. */
size_t qamw_packed_row_bytes(int d_in, int K);

/* Section 3.7 equation: log2(K)/2 + 16/d_in, plus 16/d_out when channel scales are stored. */
double qamw_bpw(int d_out, int d_in, int K, int has_channel_scales);

/* Maps the status word written by qamw_encode / qamw_calibrate to QAMW_OK or QAMW_ERR_NONFINITE. */
int qamw_status_to_error(int32_t status_word);

/* ----------------------------------------------------------------------------------------------
 * Codebook object.
 * -------------------------------------------------------------------------------------------- */

/* Uploads the K x 2 f32 codebook (host pointer) to the current device and builds the exact
 * spatial search table used by qamw_encode (Section 3.6: the Euclidean-nearest
 * codeword): the plane is cut into grid x grid cells, narrow where a Gaussian source puts its
 * codewords and widening outwards; every cell lists all codewords whose nearest-neighbour region
 * can meet the cell, so a scan of the list returns what a scan of the whole codebook returns.
 * The outermost cells reach to |z| < 16384; points beyond are scanned exhaustively.  grid = 0
 * picks a default (about 2.2 sqrt(K), at least 31, shrunk until the table fits next to the encoder's
 * other shared memory); an explicit grid must be odd and at most 255, else
 * QAMW_ERR_ARG.  Synchronous.
 * *out must be released with qamw_codebook_destroy on the same device. */
int qamw_codebook_create(const float* codebook_host, int K, int grid, qamw_codebook** out);
void qamw_codebook_destroy(qamw_codebook* cb);

/* Polar baseline codec (Section 3.5; the corollary on the Rayleigh / uniform-phase source and the
 * remark on the cut-off R_max = 8).  Amplitude |z_k| / sigma_k goes to the nearest of N_a = 2^Ba
 * Lloyd-Max levels of the unit Rayleigh density, the phase to one of N_p = 2^Bp uniform bins whose
 * centres are the odd multiples of pi / N_p; index = (phase << Ba) | amplitude, B = Ba + Bp bits.
 *
 * qamw_polar_train: the levels, by Lloyd iterations on the density (centroids from its closed-form
 * moments on [0, 8]), rounded to f32.  levels_out: host, 2^Ba floats, ascending; c_lm_out (may be
 * NULL): the normalised distortion C_LM of those f32 levels.  Host only.
 * qamw_polar_codebook: the 2^(Ba+Bp) reconstruction points level_a (cos phi_p, sin phi_p) as a K x 2
 * f32 table (host, computed in double, rounded once), i.e. the table that decoding looks up.
 * qamw_codebook_create_polar: a codebook object for this quantiser on the current device: qamw_decode
 * uses its K x 2 table like any other codebook; qamw_encode (and qamw_encode_batch) quantise with the
 * polar rule instead of the nearest-codeword search.  A point on a level threshold takes the lower
 * level, a point on a bin boundary the bin that starts there, the origin bin 0; results within f32
 * rounding of a threshold or boundary may fall on either side.  The polar encoder exists only in
 * the kernels for the common layouts (rows and metadata 32 / 16-byte aligned, d_in a multiple of 16,
 * 32 <= block <= 512, d_in <= 14336): other shapes get QAMW_ERR_SHAPE. */
int qamw_polar_train(int Ba, float* levels_out, double* c_lm_out);
int qamw_polar_codebook(const float* levels, int Ba, int Bp, float* codebook_out);
int qamw_codebook_create_polar(const float* levels_host, int Ba, int Bp, qamw_codebook** out);

/* Introspection (host values): info_out[0..5] = grid side, total candidate entries, longest
 * candidate list, number of cells with more than four candidates, overflow entries, table bytes. */
int qamw_codebook_table_info(const qamw_codebook* cb, int32_t* info_out);

/* Host-only construction of the same table, for inspection and tests (no CUDA).  map_out: four
 * floats {zmax, c0, c1, c2} of the map from a coordinate to its column (and, alike, its row):
 *     c = min(max(z, -zmax), zmax), t = c * c, column = (grid - 1) / 2 + rn(c (c0 + t (c1 + t c2)))
 * which the device evaluates in f32 with fused multiply-adds; a point within 2^-8 of a column
 * boundary (in units of columns) is covered by the lists of both neighbours.  cells_out:
 * grid*grid records of four u16, row-major (ascending candidate indices, last repeated as
 * padding; or {0xFFFF, offset, count, 0} pointing into overflow_out).  Any output pointer may
 * be NULL; info_out as above (6 values).
 * Returns QAMW_ERR_NOMEM if the table does not fit budget_bytes or a capacity. */
int qamw_search_table_build(const float* codebook_host, int K, int grid, size_t budget_bytes,
                            float* map_out, uint16_t* cells_out, size_t cells_cap,
                            uint16_t* overflow_out, size_t overflow_cap, int32_t* info_out);

/* ----------------------------------------------------------------------------------------------
 * Device-side entry points.  chan_scale (d_in floats) may be NULL = no channel scaling;
 * signs: d_in bytes of +1/-1; sigma: d_in/2 floats; all device pointers.
 * -------------------------------------------------------------------------------------------- */

/* Bytes of device scratch qamw_calibrate needs for these parameters. */
size_t qamw_calibrate_workspace_bytes(const qamw_params* p);

/* Section 3.4 equation: sigma_k = mean_i |(y_2k, y_2k+1)| / sqrt(pi/2) over n = min(d_out, 1024)
 * rows i = floor(t*d_out/n), rows of zero norm skipped, y as in the arithmetic contract above;
 * floored at 1e-4/sqrt(d_in); 1/sqrt(d_in) when no row qualifies.  The column means are
 * accumulated in double, per thread block and then in a fixed order, so the result is
 * reproducible (QAMW_FLAG_HALF_DEVICE groups the rows differently: the double sums, and rarely the
 * last bit of a sigma, can differ between the two settings).  workspace: device scratch of at least qamw_calibrate_workspace_bytes(p) bytes,
 * 8-byte aligned, overwritten.  status_out: device int32, bit 0 set if a row norm was not finite
 * (may be NULL). */
int qamw_calibrate(const void* W, const qamw_params* p, const float* chan_scale, const int8_t* signs,
                   float* sigma_out, void* workspace, size_t workspace_bytes, int32_t* status_out,
                   void* stream);

/* qamw_calibrate for callers that must not allocate device memory.  (The paper has no counterpart
 * of this entry point: it exists for the way the library is embedded, not for the method.)
 * Some hosts of this library own the whole device heap themselves, or run inside a region where
 * cudaMalloc is forbidden or would synchronise the device: an inference server with a fixed memory
 * plan, a plug-in called between two kernels of somebody else's stream.  They cannot provide the
 * scratch buffer that qamw_calibrate wants.  This variant takes the same inputs and writes the same
 * sigma_out, but keeps its partial sums in an array of QAMW_STATIC_SCRATCH_BYTES (16 MiB) that is
 * compiled into the library.  Every device that loads the library holds that array until the
 * process exits.  The call itself allocates nothing: no cudaMalloc, no cudaFree, no allocating
 * library routine.
 *   - Shapes whose scratch need (qamw_calibrate_workspace_bytes) exceeds the array are refused with
 *     QAMW_ERR_NOMEM and a message in qamw_last_cuda_error(); nothing is launched.
 *   - The first call on each device looks up the array's device address (with that device
 *     current); make that first call outside any stream capture.  Later calls only launch.
 *   - All calls on a device share the one array, and it keeps what the last call left there.  No
 *     part of it has to be zero on entry, so nothing is cleared; but two calls whose kernels may
 *     run at the same time on one device (different streams, different host threads) overwrite each
 *     other's partial sums: order them on one stream or with events.
 * Arguments, results and error codes are otherwise those of qamw_calibrate. */
int qamw_calibrate_static(const void* W, const qamw_params* p, const float* chan_scale, const int8_t* signs,
                          float* sigma_out, int32_t* status_out, void* stream);

/* Section 3.1 steps 1-6 (after Section B.2 scaling) for all rows.  The codebook must have been
 * created on the current device (QAMW_ERR_ARG otherwise; the same holds for qamw_decode).  Writes packed_out
 * [d_out, packed_row_stride] bytes, row_norm_out [d_out] f32 and ORs bit 0 into *status_out
 * (device int32, caller-zeroed, may be NULL) for non-finite rows. */
int qamw_encode(const void* W, const qamw_params* p, const float* chan_scale, const int8_t* signs,
                const float* sigma, const qamw_codebook* cb, uint8_t* packed_out, float* row_norm_out,
                int32_t* status_out, void* stream);

/* The whole encoder side in one call, with the arguments of the paper's problem statement (Section
 * 3.1 with the scaling of Section B.2): W, activation statistics, scaling exponent, block size and
 * K (in p), codebook in; packed stream, row norms and the per-matrix metadata out.  Runs
 * qamw_channel_scales and qamw_make_signs on the host (act_rms_host: host, d_in floats, or NULL; no
 * scaling when it is NULL or alpha == 0, chan_scale_out may then be NULL), copies their d_in values
 * to chan_scale_out / signs_out, then qamw_calibrate and qamw_encode on `stream`.  All other
 * pointers device; workspace as for qamw_calibrate.  The two small host-to-device copies are issued
 * on `stream` from pageable memory (the call may wait for the stream's earlier work before them).
 * Results are those of the four calls made one after the other. */
int qamw_quantize(const void* W, const qamw_params* p, const float* act_rms_host, float alpha, uint64_t sign_seed,
                  const qamw_codebook* cb, float* chan_scale_out, int8_t* signs_out, float* sigma_out,
                  uint8_t* packed_out, float* row_norm_out, void* workspace, size_t workspace_bytes,
                  int32_t* status_out, void* stream);

/* Diagnostic variant of the encoder front half: writes y (the rotated unit direction, before the
 * division by sigma) as f32 [d_out, d_in] and the row norms; used to check stage-wise parity. */
int qamw_rotate(const void* W, const qamw_params* p, const float* chan_scale, const int8_t* signs,
                float* y_out, float* row_norm_out, int32_t* status_out, void* stream);

/* Section 3.2 + B.2: W_hat[d_out, d_in] bf16 (row stride d_in) from the packed stream. */
int qamw_decode(const uint8_t* packed, const float* row_norm, const float* chan_scale,
                const int8_t* signs, const float* sigma, const qamw_codebook* cb, const qamw_params* p,
                void* w_hat_bf16_out, void* stream);

/* Variants around the path.
 * qamw_round_f16 (Section 3.2: the bitrate charges 16 bits per row norm and per channel scale; storing
 * the norm as binary16 adds a radial quantisation term): rounds n f32 values on the device,
 * in place, to IEEE binary16 (nearest even) and back.  Round channel scales and sigma before
 * qamw_encode, row norms after it, and decode sees exactly what a 16-bit serialisation would hold.
 * qamw_renorm_row_norms (Section A.3, the optional final direction renormalisation): writes
 * row_norm_out[i] = r_i / |yhat_i|, |yhat_i|^2 = sum_k sigma_k^2 |c_idx_k|^2 (the rotation preserves
 * lengths, Lemma 1); decoding with these factors in place of the row norms gives rows whose scaled
 * length is r_i again.  row_norm_out may alias row_norm.  Both asynchronous on `stream`. */
int qamw_round_f16(float* values, size_t n, void* stream);
int qamw_renorm_row_norms(const uint8_t* packed, const float* row_norm, const float* sigma, const qamw_codebook* cb,
                          const qamw_params* p, float* row_norm_out, void* stream);

/* Fused decode -> matrix-vector product (the paper's Section 1 and Limitations name the fused
 * dequantise-matmul kernel as future work; its own pipeline writes W_hat in BF16 first):
 *     y[i, v] = sum_j W_hat[i, j] x[v, j],   W_hat the decoder's output of Section 3.2 / B.2 before
 * its rounding to bf16.  Because the rotation is orthonormal and symmetric (Lemma 1),
 * w_hat_i . x = r_i sum_k c_idx_k . (sigma_k xt_k) with xt = F S (x / s): the activation is rotated once
 * per call and no row is ever rotated back or written out.
 * x: device, n_vec vectors of d_in floats (n_vec in {1, 2, 4}); y_out: device, [d_out, n_vec] floats;
 * workspace: device, qamw_gemv_workspace_bytes(p, n_vec) bytes, 8-byte aligned.  d_in must be a
 * multiple of 32 (QAMW_ERR_SHAPE).  Packed rows and x that are 16-byte aligned (base and stride) take
 * the kernel that keeps the rotated activations in registers (one launch, any d_in up to the row-length
 * limit above); any other layout, or QAMW_FLAG_GENERAL_KERNELS, takes a layout-agnostic pair of kernels
 * whose rotated activations (n_vec * d_in floats) must fit in shared memory next to the codebook
 * (QAMW_ERR_NOMEM otherwise).  f32 accumulation in a fixed order: results are reproducible run to run;
 * asynchronous on `stream`. */
size_t qamw_gemv_workspace_bytes(const qamw_params* p, int n_vec);
int qamw_decode_gemv(const uint8_t* packed, const float* row_norm, const float* chan_scale, const int8_t* signs,
                     const float* sigma, const qamw_codebook* cb, const qamw_params* p, const float* x, int n_vec,
                     float* y_out, void* workspace, size_t workspace_bytes, void* stream);

/* Measures the device's plain FP32 issue rate with a fused-multiply-add kernel (eight independent
 * chains per thread): lane instructions per second, i.e. half the FMA FLOP/s.  This is the roofline an
 * exhaustive nearest-codeword search (QAMW_FLAG_BRUTE_FORCE) is bound by; the paper gives no such
 * figure.  scratch_dev: device, one float.  Synchronous (times its own launch with events). */
int qamw_measure_fp32_peak(float* scratch_dev, double* lane_inst_per_s_out);

/* Corollary 3 / Corollary 4 sums in double:
 *   out4[0] = sum (W - W_hat)^2        out4[1] = sum W^2
 *   out4[2] = sum r_j^2 (W - W_hat)^2  out4[3] = sum r_j^2 W^2     (r_j = act_rms, 1 if NULL)
 * so that rho_w = sqrt(out4[0]/out4[1]) and the diagonal-M_x rho_o = sqrt(out4[2]/out4[3]).
 * W as described by p; W_hat bf16 with row stride d_in; out4: device, 4 doubles, overwritten. */
int qamw_distortion(const void* W, const void* w_hat_bf16, const float* act_rms, const qamw_params* p,
                    double* out4, void* stream);

/* ----------------------------------------------------------------------------------------------
 * Batches: every linear weight of a layer or of a whole model behind one handle, so that one
 * persistent launch per phase walks all matrices (Section 3.1 / 3.2 applied matrix after matrix,
 * as the paper's quantisation driver does).  The shared-memory tables are then filled once per
 * phase instead of once per matrix, which is what small matrices spend their time on otherwise.
 * -------------------------------------------------------------------------------------------- */

/* One matrix of a batch: the arguments of the single-matrix entry points, all device pointers.
 * chan_scale and act_rms may be NULL; a pointer that a phase does not use may be NULL as long as
 * that phase is never called on the batch (e.g. no W for a decode-only batch). */
typedef struct {
    qamw_params p;
    const void* W;           /* [d_out, w_row_stride] f32 or bf16 */
    const float* chan_scale; /* [d_in] or NULL */
    const int8_t* signs;     /* [d_in] */
    float* sigma;            /* [d_in/2]: written by qamw_calibrate_batch, read by encode and decode */
    const float* act_rms;    /* [d_in] or NULL: weights of the distortion sums */
    uint8_t* packed;         /* [d_out, packed_row_stride] */
    float* row_norm;         /* [d_out] */
    void* w_hat_bf16;        /* [d_out, d_in] bf16 */
    double* dist4;           /* 4 doubles */
} qamw_matrix;

typedef struct qamw_batch qamw_batch; /* opaque: validated copy of the items plus their device descriptors */

/* Validates n items (host array, copied) against the rules of the single-matrix calls and uploads
 * their descriptors to the current device, which must be the codebook's.  All items share block, K
 * and w_dtype (QAMW_ERR_ARG otherwise).  Synchronous; allocates n small descriptors on the device,
 * released by qamw_batch_destroy.  The codebook must outlive the batch. */
int qamw_batch_create(const qamw_matrix* items, int n, const qamw_codebook* cb, qamw_batch** out);
void qamw_batch_destroy(qamw_batch* b);

/* Device scratch qamw_calibrate_batch needs (the per-matrix needs, each rounded up to 256 bytes). */
size_t qamw_batch_workspace_bytes(const qamw_batch* b);

/* The four phases over all matrices of the batch, each equivalent to calling the single-matrix
 * entry point on every item in order (same results bit for bit, same error codes), asynchronous on
 * `stream`.  Matrices in the common layout (rows and metadata 16-byte aligned, d_in a multiple of
 * 16, block >= 32) are handled by one launch per phase -- up to three in calibrate and encode, whose
 * kernels run with one of three block sizes chosen by row length; if any item falls outside, the
 * phase falls back to one launch per matrix.  Two exceptions to "bit for
 * bit": the batched calibration groups the rows differently (pair scales agree to the last bits,
 * about 1e-7 relative), and the batched distortion adds its partial sums in a fixed order, so its four
 * sums are the same bits on every run (the single-matrix call uses atomic adds; both agree to about
 * 1e-15 relative).  The handle owns a little device scratch for that (partial sums, a ticket
 * counter that is zero between launches): calls on one batch must not overlap on the device, and a
 * launch that was aborted leaves the distortion phase of that handle unusable (create a new one). */
int qamw_calibrate_batch(const qamw_batch* b, void* workspace, size_t workspace_bytes, int32_t* status_out,
                         void* stream);
int qamw_encode_batch(const qamw_batch* b, int32_t* status_out, void* stream);
int qamw_decode_batch(const qamw_batch* b, void* stream);
int qamw_distortion_batch(const qamw_batch* b, void* stream);

/* Last CUDA error string seen by the library on this thread (host, static storage). */
const char* qamw_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* QAMW_H_ */
