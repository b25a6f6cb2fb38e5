/* S2A 4-bit activation stash for GELU and softmax -- C ABI of libs2a.so (sm_100a).
 *
 * The library implements the "Non-Parametric Layers" part (Section 3.2) of
 * "Structure to Activation" (arXiv 2503.08154): in the forward pass a fused kernel
 * evaluates the nonlinearity, writes its output, and keeps for the backward pass only
 * a 4-bit code per element of the one tensor the derivative needs; in the backward
 * pass a fused kernel unpacks and dequantises the codes and forms grad_in.
 *
 * Conventions shared by all four kernels
 * --------------------------------------
 * - Every pointer is a DEVICE pointer into memory the caller owns.  The library
 *   allocates nothing, creates no stream and never synchronises; each call only
 *   enqueues work on `cuda_stream` (a cudaStream_t passed as void*, NULL = the
 *   default stream) and returns.
 * - Tensors are contiguous and row-major: n_elems = n_rows * row_len.  A row is the
 *   softmax axis, and for GELU the group of row_len consecutive elements that share
 *   one quantisation range (normally the hidden vector of one token).
 * - `dt` selects the element type of x / y / grad_out / grad_in: S2A_F32 (binary32)
 *   or S2A_BF16 (bfloat16).  Arithmetic is binary32 in registers.
 * - codes: s2a_codes_bytes(n_elems) bytes.  Element e of the flat tensor owns the low
 *   nibble of byte e/2 when e is even and the high nibble when e is odd; with an odd
 *   n_elems the last high nibble is written as 0.  (The paper fixes only the bit
 *   width; the packing is this library's.)
 * - meta: two floats per row, meta[2r] = min_r and meta[2r+1] = s_r of Eq. 8.
 * - Quantiser (Eq. 8 with N = 4, per row, in correctly rounded binary32):
 *     d = max - min; s = d / 15; inv = 15 / d;
 *     code = round_half_even((v - min) * inv), a value in 0..15;
 *   a constant row (d == 0) gets codes 0 and s = 0.  Dequantiser (Eq. 9):
 *   v_hat = code * s + min.
 * - Alignment: x, y, grad_out, grad_in and codes must be 16-byte aligned, meta 8-byte
 *   aligned.  In-place use (y == x, grad_in == grad_out) is allowed; an output that
 *   overlaps its input without being the same tensor returns S2A_ERR_OVERLAP; codes and
 *   meta must not overlap any other argument (not checked).
 * - Errors: arguments are checked on the host before anything is enqueued; an argument
 *   error (every status but S2A_ERR_CUDA) launches nothing and writes nothing.
 *   S2A_ERR_CUDA means the runtime refused a launch; a call that needs two launches (full
 *   tiles, then the rows left over) may by then have enqueued the first.  n_elems == 0
 *   returns S2A_OK without a launch.  Inputs must be finite.
 * - State: the library reads no environment variable and keeps no tensor state.  What it
 *   keeps per GPU is a 4-byte error word (s2a_device_error) and, on the host, the results
 *   of one-time look-ups per device (kernel attributes, the SM count, device addresses of
 *   its own symbols).  Any thread may make the first call on a GPU; the look-ups do not
 *   survive a cudaDeviceReset of that GPU in the same process.
 * - Supported row_len: 1 .. 2^31-1 (row lengths whose rows fit a shared-memory tile
 *   take the pipelined path; others a slower row-at-a-time path).
 */
#ifndef S2A_H_
#define S2A_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum { S2A_F32 = 0, S2A_BF16 = 1 } s2a_dtype;

typedef enum {
  S2A_OK = 0,
  S2A_ERR_NULL = 1,   /* a required pointer is NULL                              */
  S2A_ERR_SHAPE = 2,  /* row_len == 0, or n_elems not a multiple of row_len      */
  S2A_ERR_ALIGN = 3,  /* a pointer is not aligned as stated above                */
  S2A_ERR_DTYPE = 4,  /* dt is neither S2A_F32 nor S2A_BF16                      */
  S2A_ERR_CUDA = 5,   /* the CUDA runtime refused the launch                     */
  S2A_ERR_DEVICE = 6, /* a kernel gave up on a bounded wait (see s2a_device_error) */
  S2A_ERR_TOO_LARGE = 7, /* beyond the built-in scratch of s2a_gelu_fwd_tensor_range_static */
  S2A_ERR_OVERLAP = 8 /* the output overlaps the input without being the same tensor   */
} s2a_status;

/* Bytes of packed codes for n_elems elements: (n_elems + 1) / 2. */
size_t s2a_codes_bytes(size_t n_elems);

/* Bytes of per-row metadata: (n_elems / row_len) * 2 * sizeof(float); 0 if row_len is 0. */
size_t s2a_meta_bytes(size_t n_elems, size_t row_len);

/* Static, human-readable name of a status code. */
const char* s2a_status_string(int status);

/* GELU forward with stash.  Eq. 10: y = x * sigmoid(1.702 x).  The stash is Eq. 8
 * applied per row to the INPUT clipped into [-2, 2] (Section 3.2, "GeLU layer").
 *   x      in   n_elems elements of type dt
 *   y      out  n_elems elements of type dt (may alias x)
 *   codes  out  s2a_codes_bytes(n_elems) bytes
 *   meta   out  s2a_meta_bytes(n_elems, row_len) bytes
 */
int s2a_gelu_fwd(const void* x, void* y, uint8_t* codes, float* meta, size_t n_elems,
                 size_t row_len, int dt, void* cuda_stream);

/* GELU backward from the stash.  Eq. 9 gives x_hat; Eq. 12 gives the derivative
 * sigmoid(1.702 x_hat) + 0.22 sin(1.5 x_hat); grad_in = grad_out * derivative.  The 16
 * derivative values a row can take are evaluated in binary64 and rounded to binary32.
 *   grad_out in   n_elems elements of type dt
 *   codes    in   as written by s2a_gelu_fwd
 *   meta     in   as written by s2a_gelu_fwd
 *   grad_in  out  n_elems elements of type dt (may alias grad_out)
 */
int s2a_gelu_bwd(const void* grad_out, const uint8_t* codes, const float* meta, void* grad_in,
                 size_t n_elems, size_t row_len, int dt, void* cuda_stream);

/* Softmax forward with stash.  Eq. 7 over each row (the row maximum is subtracted
 * first); y is rounded to dt and the values AS WRITTEN are quantised with Eq. 8 over
 * the row, so codes == Q(y) exactly.  Arguments as for s2a_gelu_fwd.
 */
int s2a_softmax_fwd(const void* x, void* y, uint8_t* codes, float* meta, size_t n_elems,
                    size_t row_len, int dt, void* cuda_stream);

/* Softmax backward from the stash.  Eq. 9 gives y_hat; the Jacobian of Eq. 7 at y_hat
 * applied to grad_out gives grad_in_i = y_hat_i * (grad_out_i - sum_j grad_out_j y_hat_j).
 * Arguments as for s2a_gelu_bwd.
 */
int s2a_softmax_bwd(const void* grad_out, const uint8_t* codes, const float* meta, void* grad_in,
                    size_t n_elems, size_t row_len, int dt, void* cuda_stream);

/* SiLU / Swish forward and backward with the same 4-bit input stash.  Section 3.2 (end of
 * the "GeLU layer" paragraph) says the design carries over to SiLU and Swish but prints no
 * constants for them, so the reading is this library's: y = x * sigmoid(x); the input is clipped into [-C, C] with
 * C = 2 * 1.702 = 3.404 (binary32), which spans the same range of the sigmoid's argument as
 * GELU's [-2, 2]; Eq. 8 / Eq. 9 per row as for GELU; the backward pass multiplies grad_out by
 * the EXACT derivative sigmoid(x_hat) * (1 + x_hat * (1 - sigmoid(x_hat))), evaluated in
 * binary64 for the 16 values a row can take.  Arguments and rules as for s2a_gelu_fwd /
 * s2a_gelu_bwd.
 */
int s2a_silu_fwd(const void* x, void* y, uint8_t* codes, float* meta, size_t n_elems, size_t row_len, int dt,
                 void* cuda_stream);
int s2a_silu_bwd(const void* grad_out, const uint8_t* codes, const float* meta, void* grad_in, size_t n_elems,
                 size_t row_len, int dt, void* cuda_stream);

/* Bytes of scratch memory s2a_gelu_fwd_tensor_range needs for n_elems elements:
 * 8 + 8 * ceil(n_elems / 65536). */
size_t s2a_tensor_range_scratch_bytes(size_t n_elems);

/* GELU forward whose stash uses ONE quantiser range for the whole tensor -- the other
 * reading of Section 3.2, "GeLU layer", which says that the clipped input is quantised over
 * its min-to-max range without saying over which elements: here Eq. 8's min and max are
 * taken over the whole clipped tensor.  y is as for s2a_gelu_fwd;
 * every row's metadata carries the same (min, s), so s2a_gelu_bwd consumes the stash
 * unchanged.  The range must be known before the first code, so x is read twice
 * (6.5 bytes per bfloat16 element instead of 4.5).  Three kernels are enqueued.
 *   x, y, codes, meta  as for s2a_gelu_fwd (y may be x itself: the range pass has finished
 *                      with x before the pass that writes y starts, and that pass reads
 *                      each element before it writes it)
 *   scratch            device memory, s2a_tensor_range_scratch_bytes(n_elems) bytes, 8-byte
 *                      aligned, owned by the caller; contents on entry are ignored, and it
 *                      must not be used by other work on the GPU until the call's kernels
 *                      have finished
 * Errors as for s2a_gelu_fwd.
 */
int s2a_gelu_fwd_tensor_range(const void* x, void* y, uint8_t* codes, float* meta, void* scratch,
                              size_t n_elems, size_t row_len, int dt, void* cuda_stream);

/* Largest n_elems s2a_gelu_fwd_tensor_range_static accepts: 536,870,912 (8192 chunks of
 * 65,536 elements). */
size_t s2a_tensor_range_static_max_elems(void);

/* s2a_gelu_fwd_tensor_range for callers that cannot hand the library any scratch memory.
 * (The paper has no counterpart to this entry point; it exists for the sake of such
 * callers only and computes exactly what s2a_gelu_fwd_tensor_range computes.)
 *
 * Who this is for: code that is not allowed to allocate device memory at the point of the
 * call -- a plug-in whose host application owns the device allocator, a serving or
 * real-time loop in which a cudaMalloc would synchronise the device and stall every other
 * stream, a program that must fix its whole memory plan before it starts -- and that has
 * no spare buffer of its own to lend.  This entry point calls no cudaMalloc, cudaFree or
 * any other allocating routine.  Its range partials go to a fixed array of 65,544 bytes
 * that is part of the library image: every GPU that loads libs2a.so holds that array from
 * load to exit, whether or not this function is ever called.
 *
 * Limits and rules:
 * - n_elems <= s2a_tensor_range_static_max_elems(); a larger tensor returns
 *   S2A_ERR_TOO_LARGE and nothing is enqueued (use the variant with caller scratch).
 * - All calls on one GPU share the one array.  It keeps whatever the previous call left;
 *   nothing in it needs to start at zero, because each call overwrites every slot it later
 *   reads.  Two calls whose kernels can run at the same time on the same GPU (different
 *   streams, different host threads) race on it and produce wrong codes: keep such calls
 *   on one stream or order them yourself.
 * - The first call on each GPU looks up the array's device address (with that GPU current);
 *   make that first call outside any stream capture.
 * - The look-up is safe from any thread; it does not survive a cudaDeviceReset of the GPU.
 * Arguments and the other errors are those of s2a_gelu_fwd_tensor_range without `scratch`.
 */
int s2a_gelu_fwd_tensor_range_static(const void* x, void* y, uint8_t* codes, float* meta, size_t n_elems,
                                     size_t row_len, int dt, void* cuda_stream);

/* Bytes of the ReLU bit mask for n_elems elements: (n_elems + 7) / 8. */
size_t s2a_mask_bytes(size_t n_elems);

/* ReLU forward with a 1-bit stash (Section 3.2, "ReLU layer": the derivative takes the
 * values 0 and 1 only).  y = x where x > 0, else +0.  Element e of the flat tensor owns bit
 * (e mod 8), least significant first, of mask byte e / 8; unused bits of the last byte are
 * written as 0.  No rows, no metadata.
 *   x     in   n_elems elements of type dt (16-byte aligned)
 *   y     out  n_elems elements of type dt (16-byte aligned, may alias x)
 *   mask  out  s2a_mask_bytes(n_elems) bytes
 */
int s2a_relu_fwd(const void* x, void* y, uint8_t* mask, size_t n_elems, int dt, void* cuda_stream);

/* ReLU backward from the mask: grad_in = grad_out where the element's bit is set, else +0.
 *   grad_out in   n_elems elements of type dt (16-byte aligned)
 *   mask     in   as written by s2a_relu_fwd
 *   grad_in  out  n_elems elements of type dt (16-byte aligned, may alias grad_out)
 */
int s2a_relu_bwd(const void* grad_out, const uint8_t* mask, void* grad_in, size_t n_elems, int dt,
                 void* cuda_stream);

/* Eq. 8 is stated for a general bit width N; these are the four kernels with N = `bits`.
 * bits = 4 is exactly s2a_gelu_fwd / _bwd / s2a_softmax_fwd / _bwd (same kernels, same
 * speed).  bits = 2 and bits = 8 use 3 and 255 quantisation levels, pack 4 codes or 1 code
 * per byte (element e owns bits [(e N) mod 8, (e N) mod 8 + N) of byte (e N) / 8, least
 * significant first).  Pipelined forms at these widths: the GELU pair for rows of whole
 * 16-byte vectors with at least 128 of them (row_len >= 1024 bfloat16, 512 binary32), the
 * softmax pair for any row_len >= 16 whose rows fit a shared-memory tile (about half the
 * bandwidth of the 4-bit kernels); other shapes run row at a time.
 * codes: s2a_codes_bytes_bits(n_elems, bits) bytes.  Any other
 * `bits` returns S2A_ERR_SHAPE.  Everything else as for the 4-bit entry points.
 */
size_t s2a_codes_bytes_bits(size_t n_elems, int bits);
int s2a_gelu_fwd_bits(const void* x, void* y, uint8_t* codes, float* meta, size_t n_elems, size_t row_len,
                      int bits, int dt, void* cuda_stream);
int s2a_gelu_bwd_bits(const void* grad_out, const uint8_t* codes, const float* meta, void* grad_in, size_t n_elems,
                      size_t row_len, int bits, int dt, void* cuda_stream);
int s2a_softmax_fwd_bits(const void* x, void* y, uint8_t* codes, float* meta, size_t n_elems, size_t row_len,
                         int bits, int dt, void* cuda_stream);
int s2a_softmax_bwd_bits(const void* grad_out, const uint8_t* codes, const float* meta, void* grad_in,
                         size_t n_elems, size_t row_len, int bits, int dt, void* cuda_stream);

/* Channel Average Pooling (Eq. 5), the parameter-free connector of the side branch.
 * x is [n_rows, channels], y is [n_rows, channels / r]: y_k = (1/r) * sum_{j<r} x_{k r + j};
 * the sum runs in index order in binary32.  No activation is kept for backward (the
 * gradient needs only r).  channels must be a multiple of r (else S2A_ERR_SHAPE); x and y
 * 16-byte aligned.
 */
int s2a_cap_fwd(const void* x, void* y, size_t n_rows, size_t channels, size_t r, int dt, void* cuda_stream);

/* Backward of Eq. 5: grad_in_{k r + j} = grad_out_k / r.  grad_out is [n_rows, channels / r],
 * grad_in is [n_rows, channels].
 */
int s2a_cap_bwd(const void* grad_out, void* grad_in, size_t n_rows, size_t channels, size_t r, int dt,
                void* cuda_stream);

/* Low-Rank Prompt forward (Eq. 3): y[b] = x[b] + A B for every sample b of a
 * [batch, tokens, channels] activation, with A [tokens, rank] and B [rank, channels] in
 * binary32 (device pointers).  The product is accumulated in binary32, k in order.  The
 * gradient to the activation (Eq. 4) is grad_out itself and needs no call.  y may alias x.
 */
int s2a_lrp_fwd(const void* x, const float* A, const float* B, void* y, size_t batch, size_t tokens,
                size_t channels, size_t rank, int dt, void* cuda_stream);

/* The pipelined kernels wait on shared-memory barriers with an iteration limit; a
 * wait that runs out records a bit in a per-device word and the kernel returns early.
 * This call copies that word of the CURRENT device into *flags (0 = no kernel ever gave
 * up) and clears it when `clear` is non-zero.  It synchronises the device.  Returns
 * S2A_OK, S2A_ERR_NULL or S2A_ERR_CUDA.
 */
int s2a_device_error(unsigned int* flags, int clear);

/* Self-test of the bounded waits.  Enqueues one warp that waits, with a 2 ms limit, for a
 * shared-memory barrier phase that nothing completes: the wait runs out, the kernel records
 * bit 2 (value 4) in the CURRENT device's error word and returns.  Afterwards
 * s2a_device_error reports 4 until it is cleared, and the context is as usable as before.
 * It lets an integrator (and this library's tests) see the give-up path work without any
 * real fault.  Bits 0 and 1 of the word belong to the pipelined kernels (a consumer gave up
 * waiting for a tile; the copy lane gave up waiting for the consumers).  Returns S2A_OK or
 * S2A_ERR_CUDA.  (The paper has no counterpart: this concerns the kernels' plumbing only.)
 */
int s2a_selftest_wait_expiry(void* cuda_stream);

/* Self-test of an assumption of the fixed-width bfloat16 softmax forward (row lengths 49, 50,
 * 64, 197, 257).  Those kernels do not search y for the range of Eq. 8: they take the row's
 * smallest and largest INPUT and send both through the same operations as every element.  That
 * equals min(y) and max(y) as written provided no operation on the way ever decreases when its
 * argument grows.  The correctly rounded ones cannot; the GPU's approximate 2^x is checked by
 * this call: it evaluates it at every binary32 argument between -150 and 1 (all the kernels can
 * produce; below -126 the result is flushed to zero), compares neighbours, and writes the
 * number of neighbouring pairs found out of order to the HOST word *out_of_order (0 on every
 * GPU this library is built for; anything else means those kernels must not be trusted there).
 * About 2.2e9 evaluations, a few milliseconds; synchronises the stream.  Returns S2A_OK,
 * S2A_ERR_NULL or S2A_ERR_CUDA.
 */
int s2a_selftest_exp2_monotone(unsigned long long* out_of_order, void* cuda_stream);

/* How a call would be run: writes into `out` (capacity `cap` bytes, always
 * NUL-terminated) a one-line description of the kernel variant and launch shape chosen
 * for (kernel, row_len, dt, n_elems).  kernel: 0 gelu_fwd, 1 gelu_bwd, 2 softmax_fwd,
 * 3 softmax_bwd, 4 silu_fwd, 5 silu_bwd.  Host-only; launches nothing.  Returns S2A_OK or an argument error.
 */
int s2a_describe_plan(int kernel, size_t n_elems, size_t row_len, int dt, char* out, size_t cap);

#ifdef __cplusplus
}
#endif
#endif /* S2A_H_ */
