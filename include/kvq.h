/*
 * kvq.h -- C ABI of libkvq: fused int4 KV-cache quantizer for NVIDIA B200 (sm_100a).
 *
 * The library quantizes head-dim vectors x in R^D to 4-bit codes plus fp16 group
 * scales and reconstructs them:
 *
 *   encode:  z = pack(F diag(s) x)            sign-randomized unitary DFT in its real
 *                                             orthogonal form (Sec. 3.1, Eq. 1-2)
 *            v = lambda (.) z                 per-channel rescale (Sec. 5.1 item 1, Sec. 7.1)
 *            sigma_j = fp16(max_{c in group j} |v_c| / 7)          (Sec. 3.2 step 3, Sec. 5.6)
 *            q_c = clamp(rint(v_c / sigma_j), -7, 7)               (Sec. 3.2 step 4)
 *            byte_i = (q_{2i+1} << 4) | (q_{2i} & 0xF)             (Sec. 3.2, nibble pack)
 *   decode:  x^ = diag(s) F^-1 unpack( q sigma / max(lambda, 1e-6) ) (Sec. 3.1; Sec. 5.1 item 1)
 *
 * Conventions
 *   - DFT kernel e^{-2 pi i k n / D}; Eq. 2 packing: z_0 = Re Y_0, z_{D/2} = Re Y_{D/2},
 *     z_k = sqrt2 Re Y_k and z_{D/2+k} = sqrt2 Im Y_k for 0 < k < D/2.
 *   - groups are `group` consecutive coordinates of z; codes use the STORED fp16 scale;
 *     rounding is half-to-even; a zero scale gives zero codes.
 *   - every data pointer is a DEVICE pointer owned by the caller unless it says "host".
 *     The library owns only the plan and the small device tables hanging off it.
 *   - calls are asynchronous on the given CUDA stream (a cudaStream_t passed as void*,
 *     NULL = default stream).  The first use of a plan on a device allocates its small tables and
 *     copies them with a blocking copy; kvq_plan_prepare does that, and the per-kernel set-up,
 *     ahead of time, after which the compute calls allocate nothing and never synchronize.
 *   - every function returns a kvq_status_t; nothing throws across the boundary.
 *     Arguments are validated on the host before any CUDA call is made.
 *   - there is no CPU fallback: without a CUDA device the compute calls return KVQ_ERR_CUDA.
 */
#ifndef KVQ_H
#define KVQ_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct kvq_plan kvq_plan_t; /* opaque, library-owned */

typedef enum {
    KVQ_OK = 0,
    KVQ_ERR_INVALID_ARG = 1,     /* null pointer, negative size, lambda table too short, pos >= T_max ... */
    KVQ_ERR_UNSUPPORTED_DIM = 2, /* D or group outside the supported set */
    KVQ_ERR_ALIGNMENT = 3,       /* a base pointer is not 16-byte aligned */
    KVQ_ERR_CUDA = 4,            /* a CUDA runtime call failed (no device, launch error ...) */
    KVQ_ERR_TIMEOUT = 5,         /* a bounded device-side wait ran out (see kvq_plan_device_status) */
    KVQ_ERR_NOMEM = 6,
    KVQ_ERR_SCRATCH_LIMIT = 7,   /* the plan needs more fixed scratch than kvq_decode_static holds */
    KVQ_ERR_RANGE = 8            /* reserved (earlier: a tensor-core decode met numbers outside its operands' range;
                                    such tiles are now decoded in fp32 by the same launch) */
} kvq_status_t;

typedef enum { KVQ_F16 = 0, KVQ_BF16 = 1 } kvq_dtype_t;

/* Which kernel family serves a call.  AUTO picks by size and shape: the matrix-vector kernel for calls of up to
 * 2048 rows (1024 for D > 128; such calls are latency-bound), beyond that the tensor-core kernel where one is built for the plan's D and
 * layout and the call's dtype, else the register FFT. */
typedef enum {
    KVQ_IMPL_AUTO = 0,
    KVQ_IMPL_FFT = 1,   /* fp32 register FFT, one thread per vector: every D, dtype and layout; no rotation */
    KVQ_IMPL_GEMM = 2,  /* tcgen05 DFT-as-GEMM.  bits = 4: encode / append and decode: D = 64, 96, 128, 160, 256 in fp16
                           and bf16; either group size.  bits = 8:
                           D <= 160 in fp16, D <= 128 in bf16; at D = 256 the decode (both types, plans without
                           a rotation) and the encode from fp16.  At most 2^31 - 1 rows per call (AUTO falls back
                           to the register FFT beyond).
                           Elsewhere the compute calls return KVQ_ERR_UNSUPPORTED_DIM. */
    KVQ_IMPL_MATVEC = 3 /* fp32 matrix-vector product with the plan's D x D table, a CTA per 8 vectors: every D, dtype
                           and layout, rotated plans included; meant for small calls, correct (and slow) at any size */
} kvq_impl_t;

/*
 * kvq_plan_create -- "kvq_plan(D, group, seed)": draws the sign diagonal s (Sec. 3.1: one random
 * sign per coordinate, fixed for the life of the plan) and fixes the radix plan of the length-D/2
 * complex FFT (Sec. 3.2 step 2; mixed radix 3 / 5 for D = 96 / 160).
 *   D      head dimension; supported: 64, 96, 128, 160, 256.
 *   group  coordinates per scale; supported: 32, or D (one scale per vector).
 *   seed   sign n is -1 when the top bit of the n-th SplitMix64 output for this seed is set.
 *   out    host pointer receiving the plan.
 * Touches no GPU: device tables are created on the first compute call, on the device that is
 * current then.  Errors: INVALID_ARG (null out), UNSUPPORTED_DIM, NOMEM.
 */
kvq_status_t kvq_plan_create(int D, int group, uint64_t seed, kvq_plan_t **out);

/*
 * kvq_plan_create_ex -- kvq_plan_create with the quantizer's base variants (Sec. 3.2 steps 3-4; Sec. 4.1 "Quantization":
 * uniform symmetric codes with one scale per head-dim vector):
 *   group  32, or D for one scale per vector ("per-token"): scales are then [N, 1] fp16.
 *   bits   4 (codes in [-7, 7], two per byte as in kvq_encode) or 8 (scale = absmax / 127, codes in [-127, 127], one
 *          two's-complement byte per value: `packed` rows are D bytes).
 * Everything else is as for kvq_plan_create, which is (group, bits = 4).  Wherever a comment of this header says
 * "[*, D/2] bytes" a plan with bits = 8 takes [*, D] bytes.  The tensor-core kernels serve either group size, and
 * bits = 8 up to D = 160 and, encode from bf16 apart, at D = 256 (see KVQ_IMPL_GEMM); elsewhere such plans run on the register-FFT and matrix-vector kernels
 * (KVQ_IMPL_GEMM is refused with UNSUPPORTED_DIM); kvq_decode_static serves group = 32, bits = 4 only.
 */
kvq_status_t kvq_plan_create_ex(int D, int group, int bits, uint64_t seed, kvq_plan_t **out);

/*
 * kvq_plan_set_rotation -- learned rotation at inference (Sec. 5.1 item 2): an orthogonal R in R^{D x D} between the
 * transform and lambda, v = lambda (.) (R z) on the way in and z^ = R^T (v^ / max(lambda, 1e-6)) on the way out.
 *   R_host   HOST pointer, [D, D] row-major fp32, copied by the call; NULL removes the rotation.  The library does not
 *            check that R is orthogonal: the inverse path applies R^T.  Training R is the caller's business.
 * The rotation is folded into the plan's D x D tables, so it costs nothing per vector in the kernels that contract
 * with those tables: the tensor-core kernels (KVQ_IMPL_GEMM; D = 256 decode then runs a dense 256 x 256 kernel) and
 * the matrix-vector kernels (KVQ_IMPL_MATVEC).  A rotated plan never takes the register FFT: AUTO uses the
 * tensor-core kernel where KVQ_IMPL_GEMM lists one for the call and the matrix-vector kernel everywhere else (every
 * layout and dtype works, large calls outside the GEMM list are slow); KVQ_IMPL_FFT and kvq_decode_static return
 * UNSUPPORTED_DIM.
 * If the plan's device tables already exist they are rewritten after a device synchronisation: call it with the
 * plan's device current and no call using the plan in flight on another thread.
 * Errors: INVALID_ARG (null plan, non-finite entry, wrong device), NOMEM, CUDA.
 */
kvq_status_t kvq_plan_set_rotation(kvq_plan_t *plan, const float *R_host /* [D, D] or NULL */);

/* Frees the plan and its device tables.  NULL is a no-op.  The caller must make sure no call
 * using the plan is still running on the GPU. */
kvq_status_t kvq_plan_destroy(kvq_plan_t *plan);

/* Copies the D signs (+1 / -1) to a HOST array, so that tests can hand the same diagonal to an
 * independent implementation. */
kvq_status_t kvq_plan_get_signs(const kvq_plan_t *plan, int8_t *host_signs /* [D] */);

/* Describes the plan: the radices of the length-D/2 complex FFT in the order they are applied
 * (host array of at least 8 ints), how many there are, and the bytes of device tables the plan
 * holds once initialised.  Any output pointer may be NULL. */
kvq_status_t kvq_plan_describe(const kvq_plan_t *plan, int *radices, int *n_radices, size_t *table_bytes);

/* Selects the kernel family for later kvq_encode / kvq_append (encode_impl) and kvq_decode
 * (decode_impl) calls on this plan.  Default: AUTO for both. */
kvq_status_t kvq_plan_set_impl(kvq_plan_t *plan, kvq_impl_t encode_impl, kvq_impl_t decode_impl);

/*
 * kvq_plan_prepare -- everything a compute call would otherwise do on its first use, done now, on the
 * device that is current: allocates the plan's device tables (a status word; two [D, D] fp32 tables
 * where a tensor-core or matrix-vector kernel serves the plan), fills them with blocking copies, and
 * sets the launch attributes (shared-memory size, occupancy look-ups) of every kernel that a call with
 * this plan and this 16-bit type can take, whichever family kvq_plan_set_impl or AUTO picks later.
 *   dtype   the type of x / out in the calls that follow; call once per type that will be used.
 * After it, kvq_encode, kvq_decode, kvq_append[_at], kvq_flush_block[_at] and kvq_calibrate_lambda on
 * this plan and type make no CUDA call besides their kernel launches (kvq_calibrate_lambda: and one
 * cudaMemsetAsync) and a query of the current device: nothing allocates, nothing blocks, and the
 * calls can be recorded into a CUDA graph without a warm call first.  Call it again after
 * kvq_plan_set_rotation (a rotated D = 256 plan decodes with another kernel).  Idempotent.
 * Errors: INVALID_ARG (null plan, unknown dtype, plan already bound to another device), NOMEM, CUDA
 * (no device: arguments are checked first).
 */
kvq_status_t kvq_plan_prepare(kvq_plan_t *plan, kvq_dtype_t dtype);

/*
 * kvq_plan_set_wait_limit -- how long the tensor-core encode kernel (D <= 160) lets its first wait run.
 * Every device-side wait in the library is bounded (about 2^22 polls, seconds of wall time) and ends in
 * a status bit instead of a hang.  This knob shortens ONE of them, the wait of the role that issues the
 * tensor-core instructions for the kernel's first operand build, a point at which that role has
 * nothing in flight: with a limit of a few polls the launch gives up at once, writes nothing, frees
 * what it holds and raises bit 2 of the status word, so that an integration can see KVQ_ERR_TIMEOUT
 * reported and cleared without a fault.
 *   polls   0 restores the default.  Takes effect for later kvq_encode / kvq_append calls on this plan.
 */
kvq_status_t kvq_plan_set_wait_limit(kvq_plan_t *plan, uint32_t polls);

/* Synchronizes the current device and returns the plan's device status word through *word
 * (host): 0 when no kernel using this plan ever gave up a bounded wait or left its number
 * range.  Bits 0-2: a bounded wait ran out (load, tensor-core commit, pipeline slot): returns
 * KVQ_ERR_TIMEOUT.  Bit 3 is reserved: no kernel raises it any longer.  The tensor-core decode kernels
 * carry q sigma / lambda and the table entries divided by lambda as fp16 operands, which cannot hold
 *   - a lambda row whose reciprocals 1 / max(lambda, 1e-6) span more than a factor of 2^8
 *     (entries at or below the 1e-6 clamp of Sec. 5.1 item 1 next to ordinary ones, for instance), or
 *   - in the dense D = 256 kernel of ROTATED plans, which has no room for the other kernels' per-row
 *     power-of-two rescue, a non-zero stored scale sigma with sigma rho outside [2^-14, 9357]
 *     (rho: the power of two at or below the row's largest reciprocal);
 * a CTA that met either decodes the tiles concerned once more at the end of the same launch, in
 * fp32 on the CUDA cores (about a hundred times slower per row), so kvq_decode is exact for every
 * lambda row and scale whichever kernel serves it, and nothing is reported.
 * Bit 4: kvq_append_at or kvq_flush_block_at found a position outside the cache in device memory and
 * wrote nothing: returns KVQ_ERR_INVALID_ARG (unless bits 0-2 are set too).
 * The word is sticky until kvq_plan_clear_device_status. */
kvq_status_t kvq_plan_device_status(kvq_plan_t *plan, uint32_t *word);

/* Synchronizes the current device and clears the plan's device status word (after the caller has dealt with what it
 * reported).  Call it with the plan's device current and no call using the plan in flight. */
kvq_status_t kvq_plan_clear_device_status(kvq_plan_t *plan);

/*
 * kvq_encode -- forward path (Sec. 3.2 steps 1-4 with the fused lambda and per-group scales of
 * Sec. 7.1) on N vectors.
 *   x        device, [N, D] row-major, fp16 or bf16 per `dtype`; 16-byte aligned.
 *   lambda   device, fp32 [n_lambda, D]; row r of x uses lambda row r / rows_per_lambda
 *            (row 0 for every r when n_lambda == 1).  Requires
 *            n_lambda * rows_per_lambda >= N when n_lambda > 1.
 *   packed   device out, [N, D/2] bytes, byte i of a row = (q[2i+1] << 4) | (q[2i] & 0xF);
 *            16-byte aligned.
 *   scales   device out, [N, D/group] fp16; 16-byte aligned.
 * N == 0 is a no-op that returns KVQ_OK without looking at the data pointers.  Errors: INVALID_ARG, ALIGNMENT, UNSUPPORTED_DIM, CUDA.
 */
kvq_status_t kvq_encode(kvq_plan_t *plan, const void *x, kvq_dtype_t dtype, int64_t N,
                        const float *lambda, int64_t n_lambda, int64_t rows_per_lambda,
                        uint8_t *packed, void *scales, void *cuda_stream);

/*
 * kvq_decode -- inverse path (Sec. 3.1: Eq. 2 undone, inverse real DFT, signs last; lambda clamped at 1e-6,
 * Sec. 5.1 item 1) on N stored vectors: the per-step full-prefix read.
 *   packed, scales, lambda as in kvq_encode (inputs here);
 *   out      device out, [N, D] row-major, fp16 or bf16 per `dtype` (round to nearest even);
 *            16-byte aligned.
 */
kvq_status_t kvq_decode(kvq_plan_t *plan, const uint8_t *packed, const void *scales, int64_t N,
                        const float *lambda, int64_t n_lambda, int64_t rows_per_lambda,
                        void *out, kvq_dtype_t dtype, void *cuda_stream);

/*
 * kvq_append -- the decode-step write (Sec. 7.2: the cache stores K/V as int4 + scales between
 * decode steps): quantizes S new vectors, one per stream, and writes them to row `pos` of
 * caches laid out packed_cache [S, T_max, D/2] and scales_cache [S, T_max, D/group].
 * Stream i uses lambda row i / streams_per_lambda (row 0 when n_lambda == 1).  No other row
 * of the caches is touched.  Requires 0 <= pos < T_max.
 */
kvq_status_t kvq_append(kvq_plan_t *plan, const void *x_new /* [S, D] */, kvq_dtype_t dtype, int64_t S,
                        const float *lambda, int64_t n_lambda, int64_t streams_per_lambda,
                        uint8_t *packed_cache, void *scales_cache, int64_t T_max, int64_t pos,
                        void *cuda_stream);

/*
 * kvq_flush_block -- the residual-window flush with the dequantized-prefix cache (Sec. 7.2: new tokens wait in a short
 * fp16 window; when it is full the block is quantized, and the already dequantized prefix is kept, so that a decode step
 * costs O(new rows) instead of O(prefix)).  Quantizes `rows` new vectors of each of S streams into rows
 * [pos0, pos0 + rows) of the int4 caches (exactly what `rows` kvq_append calls would store) and writes the dequantized
 * values of those rows (exactly what kvq_decode of the caches would give there) into the same rows of dq_cache.
 *   x_block       device, [S, rows, D] row-major, fp16 or bf16 per `dtype`; 16-byte aligned.
 *   lambda, n_lambda, streams_per_lambda, packed_cache [S, T_max, D/2], scales_cache [S, T_max, D/group]: as in kvq_append.
 *   dq_cache      device out, [S, T_max, D] of the same 16-bit type; 16-byte aligned.  Only rows [pos0, pos0 + rows) are written.
 * Requires 0 <= pos0 and pos0 + rows <= T_max.  S == 0 or rows == 0 is a no-op.  One launch on the stream when
 * S * rows <= 2048 (1024 for D > 128): the matrix-vector kernel quantizes a vector, dequantizes it from the values it
 * stored and transforms it back in the same CTA.  Larger blocks take two launches (the encode as kvq_encode picks it,
 * then a decode of the stored rows, in place on the caches: the tensor-core kernel for blocks of 64 rows and more on a
 * plan without a rotation, the matrix-vector kernel on rotated plans, else the register FFT).  The
 * window itself (holding the not yet flushed tokens in fp16) is the caller's buffer: this call is its flush.
 */
kvq_status_t kvq_flush_block(kvq_plan_t *plan, const void *x_block, kvq_dtype_t dtype, int64_t S, int64_t rows,
                             const float *lambda, int64_t n_lambda, int64_t streams_per_lambda, uint8_t *packed_cache,
                             void *scales_cache, void *dq_cache, int64_t T_max, int64_t pos0, void *cuda_stream);

/*
 * kvq_append_at, kvq_flush_block_at -- kvq_append and kvq_flush_block with the cache position held in DEVICE memory.
 * (Sec. 7.2's decode loop is dominated by dispatch at these sizes; a loop that is recorded once as a CUDA graph and
 * replayed needs every per-step value to come from memory, not from a launch argument.)
 *   pos_device / pos0_device   device, one int64_t, 8-byte aligned: the row (first row) to write.  It is read when the
 *                 kernel runs, so the same call -- or a CUDA graph that holds it -- serves successive positions once
 *                 the caller updates that word on the same stream.  A value outside [0, T_max - 1] (append) or
 *                 [0, T_max - rows] (flush) writes nothing and raises bit 4 of the plan's device status word.
 * Everything else as in kvq_append / kvq_flush_block (same stored bytes, same dequantized rows).  Both always take the
 * matrix-vector kernels, one launch whatever S and rows are (kvq_plan_set_impl is not consulted).  The first call of an
 * entry point for a given plan layout and dtype on a device allocates the plan's tables and sets the kernel's launch
 * attributes; every later one makes no CUDA call but the launch, and so can be recorded into a CUDA graph: make one call
 * of the same entry point with the same dtype outside the recording first.
 */
kvq_status_t kvq_append_at(kvq_plan_t *plan, const void *x_new /* [S, D] */, kvq_dtype_t dtype, int64_t S,
                           const float *lambda, int64_t n_lambda, int64_t streams_per_lambda, uint8_t *packed_cache,
                           void *scales_cache, int64_t T_max, const int64_t *pos_device, void *cuda_stream);
kvq_status_t kvq_flush_block_at(kvq_plan_t *plan, const void *x_block, kvq_dtype_t dtype, int64_t S, int64_t rows,
                                const float *lambda, int64_t n_lambda, int64_t streams_per_lambda, uint8_t *packed_cache,
                                void *scales_cache, void *dq_cache, int64_t T_max, const int64_t *pos0_device,
                                void *cuda_stream);

/*
 * kvq_calibrate_lambda -- static calibration of the per-channel rescale (Sec. 7.1: lambda_d = 1 / per-channel
 * maximum of the SRFT output, taken in one pass over calibration vectors).
 *   x           device, [N, D] row-major, fp16 or bf16 per `dtype`; 16-byte aligned: the calibration vectors.
 *   lambda_out  device out, fp32 [D]; 16-byte aligned: lambda_c = 1 / max_n |(M (s (.) x_n))_c|, and 1 for a channel that
 *               is zero on every vector (also for N == 0).  Used as the accumulator during the call.
 * Runs the forward tensor-core kernel with lambda = 1 and an epilogue that reduces |z| over rows, then a D-thread
 * kernel that takes reciprocals: two launches on the stream, no allocation beyond the plan's first use.  Built where
 * the tensor-core encode kernel is (KVQ_ERR_UNSUPPORTED_DIM for D = 160 with bf16).
 */
kvq_status_t kvq_calibrate_lambda(kvq_plan_t *plan, const void *x, kvq_dtype_t dtype, int64_t N, float *lambda_out,
                                  void *cuda_stream);

/*
 * kvq_decode_static -- kvq_decode for callers that may not allocate device memory.  (The paper has
 * no counterpart: this entry point exists for how the library is embedded, not for the method.)
 *
 * kvq_decode calls cudaMalloc the first time a plan is used on a device (a status word, and the
 * [D, D] fp32 table of the tensor-core kernel).  A server that gave all of HBM to its own pool, a
 * decode loop that cannot take cudaMalloc's device-wide synchronisation, or a plug-in restricted to
 * the buffers it was handed cannot make that call.  This variant runs the D = 128 fp16 tensor-core kernel in its dense
 * 128 x 128 form (kvq_decode takes one radix-2 step out of it) with those two objects in a fixed 65,792-byte block that is part of the library image (every GPU
 * context that loads the library holds it until the process exits).  It calls no cudaMalloc,
 * cudaFree or other allocating routine, on any call.
 *
 *   plan         D = 128 only; a plan with D > 128 is refused with KVQ_ERR_SCRATCH_LIMIT (its table
 *                does not fit the block), smaller D and bf16 output with KVQ_ERR_UNSUPPORTED_DIM.
 *   packed, scales, N, lambda, n_lambda, rows_per_lambda, out, cuda_stream: as in kvq_decode;
 *                dtype must be KVQ_F16.
 *   status_word  optional DEVICE pointer (4-byte aligned) to a word the caller owns: cleared on the
 *                stream, then non-zero if a bounded device-side wait ran out.  NULL keeps the word
 *                inside the block, where this library version does not expose it.
 *
 * The first call on a device looks up the block's device address; make that call before any
 * stream capture begins.  A call made while its stream is being captured records the table
 * fill in front of the decode every time, so a replayed graph never depends on what other
 * calls left in the block; and since a replay changes the block behind the host's back, every
 * call on that device after the first captured one refills the table too (a few microseconds).  N must be below 2^31 (INVALID_ARG otherwise, before anything is
 * enqueued).  The block is shared: it keeps the last call's table, which belongs to
 * one plan, and a call with a different plan rewrites it on the caller's stream before decoding.
 * Calls that can overlap on the GPU (different streams, no ordering between them) race on the
 * block and on the table: order them, or use kvq_decode.
 */
kvq_status_t kvq_decode_static(kvq_plan_t *plan, const uint8_t *packed, const void *scales, int64_t N,
                               const float *lambda, int64_t n_lambda, int64_t rows_per_lambda,
                               void *out, kvq_dtype_t dtype, uint32_t *status_word, void *cuda_stream);

/* Static, human-readable name of a status code. */
const char *kvq_status_string(kvq_status_t status);

/* Number of kernels the library has launched in this process (all plans, all streams). */
uint64_t kvq_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* KVQ_H */
