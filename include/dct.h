/*
 * dct.h -- C ABI of the B200 (sm_100a) compression library for Dynamic
 * Communication Thresholding (DCT).
 *
 * The library implements the two compression operators of the paper:
 *
 *   DCT-DP (Algorithm 1): error feedback W = W_grad + E_grad; every L
 *   iterations a threshold tau = order statistic of |W|; mask M = I(|W| >= tau);
 *   compressed gradient W_hat = W .* M (sent); error E = W - W_hat (kept).
 *
 *   DCT-MP (Algorithm 2): per sample i a threshold tau_i = order statistic of
 *   |X_act,i|; mask m_i = I(|X_act,i| >= tau_i); X_act .* M and M are sent in
 *   the forward pass, X_grad .* M (same mask) in the backward pass.
 *
 * Conventions common to every entry point
 *   - Unless a parameter says "host", every pointer is a DEVICE pointer that
 *     the caller owns.  The library allocates nothing and keeps no state
 *     between calls -- with one exception, dct_dp_compress_static, whose scratch
 *     is an array built into the library (see there).
 *   - Every call is asynchronous on `stream` (a cudaStream_t passed as an
 *     opaque pointer; NULL is the legacy default stream).  No call
 *     synchronises with the host, except the *_host convenience calls.
 *   - The return value reports what the host can see before launching
 *     (arguments, workspace size, launch errors).  Conditions only the device
 *     can see (output capacity exceeded, a bounded device-side wait giving up,
 *     an out-of-range mask column) are written to `result->status` once the
 *     stream reaches that point.
 *   - Magnitudes are ordered by key(x) = bit pattern of x with the sign bit
 *     cleared, compared as an unsigned integer (uint32 for fp32, uint16 for
 *     bf16).  For non-NaN x this is the order of |x| with -0 == +0.  Ties in
 *     key are broken by the lower index / column.
 *   - Inputs are expected to be finite.  Inf orders above every finite
 *     magnitude.  NaN never traps and never causes an out-of-bounds access,
 *     but is outside the contract: the DP calls order it above Inf, while
 *     dct_mp_topk_pack_fwd may return an arbitrary (valid, k columns) selection
 *     for a row that contains NaN.
 */
#ifndef DCT_H_
#define DCT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(_WIN32)
#define DCT_API
#else
#define DCT_API __attribute__((visibility("default")))
#endif

typedef enum {
  DCT_OK              = 0,
  DCT_ERR_INVALID_ARG = 1, /* host: null pointer, k == 0, k > n, d > 32768, n > 2^31-1, aliasing */
  DCT_ERR_WORKSPACE   = 2, /* host: workspace_bytes below dct_*_workspace_bytes(n), or misaligned */
  DCT_ERR_UNSUPPORTED = 3, /* host: dtype or shape outside the supported set */
  DCT_ERR_CUDA        = 4, /* host: a CUDA runtime call failed (see dct_last_cuda_error) */
  DCT_ERR_CAPACITY    = 5, /* device: survivors > capacity; output truncated, the rest kept in the residual */
  DCT_ERR_TIMEOUT     = 6, /* device: a bounded device-side wait gave up; outputs are incomplete */
  DCT_ERR_BAD_MASK    = 7  /* device: a mask column >= d (or a packed index outside the vector) was met; that slot was skipped */
} dct_status_t;

typedef enum { DCT_F32 = 0, DCT_BF16 = 1 } dct_dtype_t;

/* cudaStream_t, passed opaquely so that this header needs no CUDA header. */
typedef void* dct_stream_t;

/* Result block in DEVICE memory, written by the kernels of one call. */
typedef struct {
  uint32_t status;   /* DCT_OK, DCT_ERR_CAPACITY, DCT_ERR_TIMEOUT or DCT_ERR_BAD_MASK */
  uint32_t reserved;
  uint64_t count;    /* compress: survivors written (<= capacity) */
  uint64_t needed;   /* compress: survivors found (may exceed capacity) */
  uint64_t n_gt;     /* select: #{ |w| >  tau } */
  uint64_t n_eq;     /* select: #{ |w| == tau };  n_gt < k <= n_gt + n_eq */
} dct_result_t;

/* Human-readable name of a status code (static storage, never NULL). */
DCT_API const char* dct_status_string(dct_status_t s);

/* Text of the last CUDA runtime error seen by this thread inside the library. */
DCT_API const char* dct_last_cuda_error(void);

/* Bytes of device workspace the calls below need for a vector of n elements.
 * The workspace must be 256-byte aligned; its contents need not be preserved
 * between calls and two calls that may overlap on the GPU need separate ones.
 * (Select: about 100 KB, from 2^25 elements on plus 4 B per element up to 32 MiB;
 * compress: 256 B plus 8 B per 4096 elements.) */
DCT_API size_t dct_threshold_select_workspace_bytes(uint64_t n);
DCT_API size_t dct_dp_compress_workspace_bytes(uint64_t n);

/*
 * dct_threshold_select -- Algorithm 1, "Error Feedback", "Sort(|W_grad|)" and
 * "Assign tau" steps (the branch taken when L divides the iteration number).
 *
 * Computes tau = the k-th LARGEST value of |fl32(grad[i] + residual[i])|,
 * i.e. the order statistic that leaves exactly k survivors when there are no
 * ties.  (The paper's tau = w_floor(N*eta) of the ascending sort with eta the
 * fraction dropped corresponds to k = N - floor(N*eta).)  Nothing is modified
 * except the outputs.
 *
 *   grad      [n] fp32, read-only.
 *   residual  [n] fp32, read-only, or NULL for E_grad = 0.
 *   n, k      1 <= k <= n <= 2^31-1.
 *   tau_out   1 fp32 (device): the threshold, sign bit clear.
 *   result    device block; n_gt, n_eq and status are written.
 *   workspace >= dct_threshold_select_workspace_bytes(n), 256-byte aligned.
 *
 * grad (and residual) should be 16-byte aligned or sit the same 4, 8 or 12
 * bytes past a 16-byte boundary (the up to three elements before them in
 * their 16-byte unit are then read); other alignments take scalar loads.
 *
 * Returns DCT_OK after enqueueing; DCT_ERR_INVALID_ARG / DCT_ERR_WORKSPACE /
 * DCT_ERR_CUDA without having launched anything.
 */
DCT_API dct_status_t dct_threshold_select(
    const float* grad, const float* residual, uint64_t n, uint64_t k,
    float* tau_out, dct_result_t* result,
    void* workspace, size_t workspace_bytes, dct_stream_t stream);

/*
 * dct_dp_compress -- Algorithm 1, "Error Feedback", "Compute mask", "Compute
 * compressed gradient", "Compute error" and the payload of "Send" for a fixed
 * threshold (the branch that reuses tau from an earlier iteration, or the one
 * that follows dct_threshold_select on the same stream).
 *
 * For every i:  w = fl32(grad[i] + residual[i]);
 *   pass(i) = key(w) > key(*tau)  ||  (key(w) == key(*tau) && fewer than
 *             *tie_budget earlier elements had key == key(*tau));
 *   with tie_budget == NULL the second clause is simply key(w) == key(*tau),
 *   which is the paper's M = I(|W| >= tau).
 * Survivors are written in ascending i as (idx_out[j], val_out[j]) = (i, w)
 * while j < capacity; residual[i] becomes +0.0 for an element that was written
 * and w for every other element, so  sent + residual == grad + old residual
 * holds for every i even when the capacity is exceeded.
 *
 *   grad       [n] fp32, read-only; must not overlap residual.
 *   residual   [n] fp32, in/out.
 *   n          1 <= n <= 2^31-1.
 *   tau        1 fp32 (device); its magnitude is used.
 *   tie_budget 1 uint64 (device) or NULL.  Passing k - n_gt from a select on
 *              the same vector yields exactly k survivors.
 *   idx_out    [capacity] int32;  val_out [capacity] fp32.  Entries at and
 *              beyond result->count are left untouched.
 *   result     device block; count, needed and status (DCT_OK,
 *              DCT_ERR_CAPACITY or DCT_ERR_TIMEOUT) are written.
 *   workspace  >= dct_dp_compress_workspace_bytes(n), 256-byte aligned.
 *
 * grad and residual should be 16-byte aligned, or sit the same 4, 8 or 12
 * bytes past a 16-byte boundary (views at one element offset into two flat
 * buffers; the up to three elements before them in their 16-byte unit are
 * then read, never written); other alignments are accepted and take a slower
 * scalar path.
 */
DCT_API dct_status_t dct_dp_compress(
    const float* grad, float* residual, uint64_t n,
    const float* tau, const uint64_t* tie_budget,
    int32_t* idx_out, float* val_out, uint64_t capacity,
    dct_result_t* result,
    void* workspace, size_t workspace_bytes, dct_stream_t stream);

/*
 * dct_mp_topk_pack_fwd -- Algorithm 2, forward pass: for every sample (row) i
 * sort |X_act,i|, take tau_i, build m_i, and pack X_act .* M together with M.
 *
 * Keeps exactly k columns per row: every column whose key exceeds key(tau_i),
 * then the lowest columns with key == key(tau_i) until k are kept, where tau_i
 * is the k-th largest magnitude of the row.
 *
 *   x_act    [rows, ld] row-major, dtype fp32 or bf16, read-only; only the
 *            first d columns of a row are looked at.
 *   rows     >= 1;  1 <= k <= d <= 32768;  ld >= d (elements).
 *   cols_out [rows*k] int16: kept columns, ascending within a row.  This IS
 *            the mask M; hand it unchanged to dct_mp_pack_bwd.
 *   vals_out [rows*k] dtype of x_act: x_act[i, cols_out[i*k+s]] (bit copies).
 *   rows_out [rows*k] int32 or NULL: explicit row id of each slot for callers
 *            that want (row, col, val) triples; the row is otherwise slot / k.
 *   tau_out  [rows] dtype of x_act or NULL: the thresholds tau_i (sign clear).
 *   result   device block or NULL; status is written (DCT_OK; see below).
 *
 * x_act rows should start on 16-byte boundaries (base aligned and ld*size a
 * multiple of 16); other layouts are accepted and take a slower scalar load.
 * Every shape gives the same result; the time does depend on it.  Rows on
 * 16-byte boundaries with d*size a multiple of 16 are packed by one warp per
 * row (bf16: d <= 8192 for k up to about d/10 and 441, d <= 3072 for k up
 * to 3d/8 and 2048; fp32: d <= 4096, k up to about d/10 and 441, denser k for
 * d <= 512) or by one CTA per row (bf16 rows of 3073..32768 columns with k
 * up to 3d/8 where the warp kernel does not apply; fp32 rows of
 * 513..32768 columns that the warp kernels leave out, k up to 3d/8);
 * short rows are held in registers, several rows to a warp (bf16 up to 128
 * columns and fp32 up to 256: every k; bf16 up to 512 columns: k up to d/8;
 * rows of up to 1024 columns at any width, stride and address: every k).
 * Everything else (denser k on longer rows, longer rows at odd strides,
 * cols_out not 4-byte aligned for the denser and the wide cases) takes a
 * general kernel that is several times slower.  status may also be DCT_ERR_TIMEOUT if a
 * bounded wait for an asynchronous copy gave up (not seen in practice; the
 * outputs are then incomplete).
 */
DCT_API dct_status_t dct_mp_topk_pack_fwd(
    const void* x_act, dct_dtype_t dtype,
    uint32_t rows, uint32_t d, uint32_t ld, uint32_t k,
    int16_t* cols_out, void* vals_out, int32_t* rows_out, void* tau_out,
    dct_result_t* result, dct_stream_t stream);

/*
 * dct_mp_pack_bwd -- Algorithm 2, backward pass: X_grad .* M packed through
 * the mask of the forward pass:  gvals_out[i*k+s] = x_grad[i, cols[i*k+s]].
 *
 *   x_grad    [rows, ld] row-major, dtype fp32 or bf16, read-only.
 *   cols      [rows*k] int16 from dct_mp_topk_pack_fwd, read-only.
 *   gvals_out [rows*k] dtype of x_grad.
 *   result    device block or NULL; status is DCT_OK, or DCT_ERR_BAD_MASK if
 *             some column was outside [0, d) (that slot is written as zero and
 *             nothing out of bounds is read).
 */
DCT_API dct_status_t dct_mp_pack_bwd(
    const void* x_grad, dct_dtype_t dtype,
    uint32_t rows, uint32_t d, uint32_t ld, uint32_t k,
    const int16_t* cols, void* gvals_out,
    dct_result_t* result, dct_stream_t stream);

/*
 * dct_dp_compress_batched -- dct_dp_compress for all the layers of a model at once.  The paper applies
 * DCT-DP layer by layer, every layer with its own threshold and its own error (Sec. 2.1); its layers
 * hold 10^3..10^6 parameters, for which one set of launches per layer costs more than the work itself.
 * This call runs every layer of `layers` -- each exactly as dct_dp_compress would -- with one reset
 * kernel, one streaming kernel over all full tiles of all 16-byte aligned layers and one kernel for
 * the ragged last tiles and the unaligned layers.
 *
 *   layers     HOST array of num_layers descriptions; the device pointers inside follow the rules of
 *              dct_dp_compress.  The array is read before the call returns.  Layers must not share
 *              residual, output or result buffers.
 *   workspace  DEVICE, >= dct_dp_compress_batched_workspace_bytes(sizes, num_layers), 256-byte aligned.
 * Every layer's result block receives its own count / needed / status.
 * Returns DCT_ERR_UNSUPPORTED while `stream` is being captured into a CUDA graph (the call uploads a table it
 * builds from `layers` on the host, which a graph would outlive).
 */
typedef struct {
  const float* grad;           /* [n] device */
  float* residual;             /* [n] device, in/out */
  uint64_t n;
  const float* tau;            /* device scalar */
  const uint64_t* tie_budget;  /* device scalar or NULL */
  int32_t* idx_out;            /* [capacity] device */
  float* val_out;              /* [capacity] device */
  uint64_t capacity;
  dct_result_t* result;        /* device */
} dct_dp_layer_t;
DCT_API size_t dct_dp_compress_batched_workspace_bytes(const uint64_t* n /* host, per layer */, uint32_t num_layers);
DCT_API dct_status_t dct_dp_compress_batched(
    const dct_dp_layer_t* layers /* host */, uint32_t num_layers,
    void* workspace, size_t workspace_bytes, dct_stream_t stream);

/*
 * dct_threshold_select_batched -- dct_threshold_select for all the layers of a model at once: the other
 * half of the layer-wise scheme of Sec. 2.1 (every L iterations each layer gets a new threshold of its
 * own).  Three streaming passes over all layers together -- every CTA works through a contiguous run of
 * 8192-element chunks and keeps the digit histogram of the layer it is in -- each followed by one small
 * kernel that scans every layer's histogram: seven launches whatever the number of layers.
 *
 * For every layer l:  *layers[l].tau_out = layers[l].k-th largest |fl32(grad + residual)| of that layer,
 * and layers[l].result->n_gt / n_eq / status are filled as by dct_threshold_select.
 *
 *   layers     HOST array of num_layers descriptions (device pointers inside; residual may be NULL;
 *              1 <= k <= n <= 2^31-1 per layer, and the sizes must add up to less than 2^44).  Read before the
 *              call returns.  Layers must not share tau_out or result.
 *   workspace  DEVICE, >= dct_threshold_select_batched_workspace_bytes(num_layers), 256-byte aligned.
 * Errors: DCT_ERR_INVALID_ARG / DCT_ERR_WORKSPACE as for dct_threshold_select, before anything is launched;
 * DCT_ERR_UNSUPPORTED while `stream` is being captured into a CUDA graph (the call uploads a table it builds
 * from `layers` on the host, which a graph would outlive).
 */
typedef struct {
  const float* grad;           /* [n] device, read only */
  const float* residual;       /* [n] device, read only, or NULL */
  uint64_t n;
  uint64_t k;
  float* tau_out;              /* device scalar */
  dct_result_t* result;        /* device */
} dct_select_layer_t;
DCT_API size_t dct_threshold_select_batched_workspace_bytes(uint32_t num_layers);
DCT_API dct_status_t dct_threshold_select_batched(
    const dct_select_layer_t* layers /* host */, uint32_t num_layers,
    void* workspace, size_t workspace_bytes, dct_stream_t stream);

/*
 * dct_dp_select_compress -- Algorithm 1 with threshold life-span L = 1: the branch "L divides the
 * iteration number" taken at every iteration, i.e. top-K sparsification with error feedback where the
 * threshold comes from the very vector that is compressed (the scheme the paper starts from, and on
 * its CPUs found 11 % slower end to end than no compression).
 *
 * The result is that of dct_threshold_select on fl32(grad + residual) followed by dct_dp_compress with the
 * tie budget k - n_gt: exactly min(k, capacity) elements are sent, the lowest indices first among those
 * equal to the threshold.  From 2^25 elements, with k small against n, the vector is streamed only once
 * (12 bytes per element, the cost of an iteration with a fixed threshold): a bound from a sector-wise
 * sample, one compress pass that leaves w in the residual and packs the elements above the bound, the
 * exact select over those, and a pass over them that sends the survivors and puts the others back; should
 * the sample misjudge the vector, the plain select and compress run on w instead (same result, decided on
 * the device).  Smaller vectors and dense k take the two operators back to back (20 bytes per element).
 *
 *   grad, residual, n, idx_out, val_out, capacity   as in dct_dp_compress.
 *   k          survivors wanted, 1 <= k <= n.
 *   tau_out    1 fp32 (device): the threshold that was used.
 *   result     device block: count (= min(k, capacity)), needed (= k), status as in dct_dp_compress,
 *              and n_gt, n_eq of the select.
 *   workspace  >= dct_dp_select_compress_workspace_bytes(n), 256-byte aligned (from 2^25 elements it includes
 *              32 MiB for the packed elements above the bound).
 */
DCT_API size_t dct_dp_select_compress_workspace_bytes(uint64_t n);
DCT_API dct_status_t dct_dp_select_compress(
    const float* grad, float* residual, uint64_t n, uint64_t k,
    float* tau_out, int32_t* idx_out, float* val_out, uint64_t capacity,
    dct_result_t* result,
    void* workspace, size_t workspace_bytes, dct_stream_t stream);

/*
 * dct_dp_decompress -- the receiving end of Algorithm 1's "Send W_hat": the sparse compressed gradient
 * goes back into a dense vector (the paper counts this decompression in the overhead of the scheme,
 * Sec. 2, without prescribing a procedure).
 *
 *   idx, val  [capacity] the packed gradient written by dct_dp_compress (ascending, distinct indices).
 *   packed    the device result block of that dct_dp_compress call; packed->count entries are used
 *             (at most `capacity`), so no host round trip is needed between the two calls.
 *   dense     [n] fp32.  accumulate == 0: dense becomes W_hat (zero everywhere else; the call clears
 *             it).  accumulate != 0: dense[idx[j]] += val[j], for a server that sums the messages
 *             of several trainers into one vector.
 *   result    device block; status is DCT_OK, or DCT_ERR_BAD_MASK if an index was outside [0, n)
 *             or the indices were not ascending (such entries are skipped, nothing out of bounds
 *             is touched).
 */
DCT_API dct_status_t dct_dp_decompress(
    const int32_t* idx, const float* val, const dct_result_t* packed, uint64_t capacity,
    float* dense, uint64_t n, int accumulate,
    dct_result_t* result, dct_stream_t stream);

/*
 * dct_mp_unpack -- the receiving end of Algorithm 2's two "send" steps: rebuilds the dense
 * [rows, ld] matrix X .* M from the mask and the packed values (X_act .* M on the next worker in the
 * forward pass, X_grad .* M on the previous worker in the backward pass).
 *
 *   cols      [rows*k] int16: the mask written by dct_mp_topk_pack_fwd.
 *   vals      [rows*k] packed values (vals_out of the forward call or gvals_out of the backward call).
 *   dense_out [rows, ld], dtype fp32 or bf16: columns 0..d-1 of every row are written (zero outside the
 *             mask); columns d..ld-1 are left untouched.
 *   result    device block or NULL; status is DCT_OK, or DCT_ERR_BAD_MASK if a column was >= d
 *             (that slot is skipped).
 */
DCT_API dct_status_t dct_mp_unpack(
    const int16_t* cols, const void* vals, dct_dtype_t dtype,
    uint32_t rows, uint32_t d, uint32_t ld, uint32_t k,
    void* dense_out, dct_result_t* result, dct_stream_t stream);

/*
 * Host-buffer convenience calls: the same operators for a caller whose data
 * lives in HOST memory (pinned memory gives full copy speed; pageable memory
 * works).  Each call copies its inputs to the caller-provided device staging
 * buffers, runs the device entry point above, copies the packed result back
 * and waits for the stream before returning.
 *
 * dct_dp_compress_host: one DCT-DP iteration for a host gradient.  The
 * residual stays resident on the device (it is state carried across
 * iterations).
 *   grad_host        [n] fp32, host.
 *   grad_dev         [n] fp32 device staging buffer.
 *   residual_dev, tau_dev, tie_budget_dev, idx_dev, val_dev, result_dev,
 *   workspace        as in dct_dp_compress (device).
 *   idx_host/val_host [capacity] host buffers receiving the first count pairs.
 *   result_host      host copy of the result block.
 * Returns the host-visible status, or the device-reported status of the call.
 */
DCT_API dct_status_t dct_dp_compress_host(
    const float* grad_host, float* grad_dev, float* residual_dev, uint64_t n,
    const float* tau_dev, const uint64_t* tie_budget_dev,
    int32_t* idx_dev, float* val_dev, uint64_t capacity,
    int32_t* idx_host, float* val_host,
    dct_result_t* result_dev, dct_result_t* result_host,
    void* workspace, size_t workspace_bytes, dct_stream_t stream);

/*
 * dct_threshold_select_host: threshold select for a host gradient (residual,
 * if any, resident on the device).  tau stays on the device for the compress
 * calls that follow; tau_host (optional) and result_host receive copies.
 */
DCT_API dct_status_t dct_threshold_select_host(
    const float* grad_host, float* grad_dev, const float* residual_dev, uint64_t n, uint64_t k,
    float* tau_dev, float* tau_host, dct_result_t* result_dev, dct_result_t* result_host,
    void* workspace, size_t workspace_bytes, dct_stream_t stream);

/*
 * dct_mp_pack_host: forward top-k pack of a host activation matrix followed by
 * the backward pack of a host gradient matrix through the same mask.
 *   x_act_host/x_grad_host [rows, ld] host; x_act_dev/x_grad_dev device staging.
 *   cols_dev/vals_dev/gvals_dev [rows*k] device; cols_host/vals_host/gvals_host
 *   [rows*k] host buffers receiving the packed results.
 */
DCT_API dct_status_t dct_mp_pack_host(
    const void* x_act_host, const void* x_grad_host, void* x_act_dev, void* x_grad_dev,
    dct_dtype_t dtype, uint32_t rows, uint32_t d, uint32_t ld, uint32_t k,
    int16_t* cols_dev, void* vals_dev, void* gvals_dev,
    int16_t* cols_host, void* vals_host, void* gvals_host,
    dct_result_t* result_dev, dct_result_t* result_host, dct_stream_t stream);

/*
 * dct_dp_compress_static -- dct_dp_compress without a workspace argument.
 * (The paper has no counterpart for this call; it exists for integration reasons only.)
 *
 * Some callers have no device memory of their own to offer as a workspace and may not obtain any:
 * a gradient hook that runs inside a framework whose caching allocator already owns the whole GPU
 * (a raw cudaMalloc there can fail outright, and it stalls every stream of the device while it
 * runs), or a plug-in that is only ever handed the tensors it must transform.  For them the tile
 * descriptors live in an array that is part of the library image itself: 262,656 bytes of device
 * memory on every GPU that loads the library, held until the process exits.  The call allocates
 * nothing -- no cudaMalloc, no cudaFree, no library routine that allocates.
 *
 * Arguments, outputs, result codes and semantics are exactly those of dct_dp_compress, with
 *   n <= DCT_DP_COMPRESS_STATIC_MAX_N (2^27 elements); a larger n returns DCT_ERR_UNSUPPORTED
 *   before anything is launched.
 * The first call on each device looks up the device address of the built-in array (with that
 * device current) and remembers it; make that first call outside any stream capture.
 * All calls on one device share the one array.  Each call re-initialises the part it uses, so
 * calls that follow one another on a stream are independent of what the previous one left
 * behind; two calls that may run on the GPU at the same time (different streams, no ordering)
 * would overwrite each other's descriptors -- use dct_dp_compress with separate workspaces then.
 */
#define DCT_DP_COMPRESS_STATIC_MAX_N (1u << 27)
DCT_API dct_status_t dct_dp_compress_static(
    const float* grad, float* residual, uint64_t n,
    const float* tau, const uint64_t* tie_budget,
    int32_t* idx_out, float* val_out, uint64_t capacity,
    dct_result_t* result, dct_stream_t stream);

/*
 * dct_threshold_select_shard_{begin,pass,advance} -- the threshold steps of Algorithm 1 (error feedback, sort,
 * assign tau) for ONE gradient vector that is range-partitioned over several GPUs: every rank holds a contiguous
 * shard of W_grad and of E_grad, and all ranks want the k-th largest |fl32(W_grad + E_grad)| of the WHOLE vector.
 * The paper's trainers each compress their own layers (Sec. 2.1) and need no such exchange; this serves a layer
 * that is itself split over GPUs.
 *
 * The select is a radix select in three passes (11 / 10 / 10 key bits).  Per pass every rank calls `pass`, which
 * writes the 2048-bin digit histogram of its own shard (restricted to the digits chosen so far) to hist_out; the
 * caller sums the histograms over the ranks (an all-reduce of 16 KiB by whatever transport it uses: the library
 * never touches another GPU's memory); every rank then calls `advance` with the summed histogram and arrives at
 * the same digit.  After advance(pass = 2) every rank's tau_out, result->n_gt and result->n_eq are those of
 * dct_threshold_select on the concatenated vector.  Compression needs no exchange: each rank runs dct_dp_compress
 * on its shard with that tau.
 *
 *   k_global   1 <= k_global <= total number of elements over all ranks (not checked: the ranks' sizes are not
 *              known here; with a larger k the outputs are unspecified).
 *   workspace  DEVICE, >= dct_threshold_select_shard_workspace_bytes(), 256-byte aligned: the state of one select
 *              (the same on every rank after every advance).  `begin` resets it.
 *   grad, residual  [n_local] fp32 device, read only; residual may be NULL; n_local may be 0 (an empty shard).
 *   pass       0, 1, 2, in this order, each followed by its advance.
 *   hist_out   [2048] uint64 DEVICE: overwritten with this shard's histogram.
 *   hist_global [2048] uint64 DEVICE: the sum over all ranks.
 *   tau_out, result  device; written by advance(pass = 2) only (may be NULL for passes 0 and 1).
 * Errors: DCT_ERR_INVALID_ARG / DCT_ERR_WORKSPACE before anything is launched.
 */
DCT_API size_t dct_threshold_select_shard_workspace_bytes(void);
DCT_API dct_status_t dct_threshold_select_shard_begin(
    uint64_t k_global, void* workspace, size_t workspace_bytes, dct_stream_t stream);
DCT_API dct_status_t dct_threshold_select_shard_pass(
    const float* grad, const float* residual, uint64_t n_local, uint32_t pass,
    const void* workspace, uint64_t* hist_out, dct_stream_t stream);
DCT_API dct_status_t dct_threshold_select_shard_advance(
    const uint64_t* hist_global, uint32_t pass, void* workspace,
    float* tau_out, dct_result_t* result, dct_stream_t stream);

/*
 * dct_threshold_select_shard_sampled_{begin,pass,advance} -- the same select with ONE streaming pass over the shard
 * instead of three, for large vectors (the scheme of dct_threshold_select carried over to shards): a sample of the
 * vector, taken at the same rate on every rank, is radix-selected in two passes for a rank chosen six standard
 * deviations on the safe side (stages 0 and 1), which gives a key `lo` with, almost surely, between k_global and a
 * few k_global elements of the whole vector at or above it; every rank streams its shard once and keeps its keys
 * >= lo (stage 2; its message is the number of keys kept and whether they fitted); the three exact passes then run
 * over the candidates only (stages 3, 4, 5) -- or, if the summed counts say that the candidates are fewer than
 * k_global or overflowed some rank's buffer, over the shards: every rank takes that decision alike.  Six stages of
 * (pass, sum of 2048 uint64 over the ranks, advance); the outputs are those of the three-pass version, bit for bit.
 *
 *   begin      returns DCT_ERR_UNSUPPORTED (nothing launched) where the scheme does not apply: n_global < 2^25, or a
 *              k_global so large that the candidates might not fit one rank's buffer of 2^22 keys; use the
 *              three-pass entry points then.  Every rank gets the same answer (it depends on k_global and n_global
 *              only).
 *   n_global   total number of elements over all ranks; n_local this rank's (may be 0).
 *   workspace  DEVICE, >= dct_threshold_select_shard_sampled_workspace_bytes(n_local), 256-byte aligned (up to
 *              16 MiB of candidate keys).
 *   stage      0 .. 5, in this order, each pass followed by its advance.
 *   hist_out / hist_global  [2048] uint64 DEVICE, as above.
 *   tau_out, result  device; written by advance(stage = 5) only.
 */
DCT_API size_t dct_threshold_select_shard_sampled_workspace_bytes(uint64_t n_local);
DCT_API dct_status_t dct_threshold_select_shard_sampled_begin(
    uint64_t k_global, uint64_t n_global, uint64_t n_local, void* workspace, size_t workspace_bytes,
    dct_stream_t stream);
DCT_API dct_status_t dct_threshold_select_shard_sampled_pass(
    const float* grad, const float* residual, uint64_t n_local, uint32_t stage,
    void* workspace, uint64_t* hist_out, dct_stream_t stream);
DCT_API dct_status_t dct_threshold_select_shard_sampled_advance(
    const uint64_t* hist_global, uint32_t stage, void* workspace,
    float* tau_out, dct_result_t* result, dct_stream_t stream);

/* ------------------------------------------------------------------------- *
 * Threshold diagnostics: the quantities behind the paper's threshold plots.
 * None of them changes a gradient, a residual or an activation.
 * ------------------------------------------------------------------------- */

#define DCT_DIAG_MAX_QUANTILES 4u

/*
 * dct_threshold_select_multi -- the top-k thresholds of one gradient vector at
 * several sparsity levels at once (Sec. 2.1, the figure that plots the top-K
 * threshold at 75 / 90 / 95 % sparsity over the iterations and motivates the
 * threshold life-span L).
 *
 * For every q < m:  tau_out[q] = ks[q]-th largest |fl32(grad + residual)|, exactly
 * as dct_threshold_select would return it for k = ks[q], with
 * results[q].n_gt / n_eq / status filled the same way.  All m thresholds come
 * out of the same three streaming passes over the vector (one shared histogram
 * of the leading digit, then one histogram per threshold), so the cost does not
 * grow with m and does not depend on how dense the quantiles are.
 *
 *   grad, residual  [n] fp32 device, read only; residual may be NULL.
 *   ks              [m] HOST array of survivor targets, 1 <= ks[q] <= n, any order.
 *   m               1 .. DCT_DIAG_MAX_QUANTILES.
 *   tau_out         [m] fp32 device.   results  [m] dct_result_t device.
 *   workspace       device, 256-byte aligned,
 *                   >= dct_threshold_select_multi_workspace_bytes(n, m); caller owned.
 * Errors: as dct_threshold_select (DCT_ERR_INVALID_ARG also for m out of range).
 */
DCT_API size_t dct_threshold_select_multi_workspace_bytes(uint64_t n, uint32_t m);
DCT_API dct_status_t dct_threshold_select_multi(
    const float* grad, const float* residual, uint64_t n,
    const uint64_t* ks, uint32_t m,
    float* tau_out, dct_result_t* results,
    void* workspace, size_t workspace_bytes, dct_stream_t stream);

/*
 * dct_mp_threshold_mean -- the mean over the batch of the per-sample top-k
 * thresholds, (1/B) sum_i tau_i, at several sparsity levels, measured without
 * sparsifying anything (Sec. 2.2, the figure that plots this mean at 75 / 90 /
 * 95 % sparsity with and without DCT-MP).
 *
 * For every q < m and row i:  tau_out[q*rows + i] = ks[q]-th largest |x[i, :d]|
 * (the tau_i of dct_mp_topk_pack_fwd for k = ks[q], bit for bit), and
 * mean_out[q] = (sum_i tau_out[q*rows + i]) / rows in binary64.  The sum is
 * accumulated in binary64 in a fixed order (the same input always gives the same
 * bits); it is the exact sum whenever that is representable, which holds for
 * every batch whose thresholds span fewer than 53 - 24 - log2(rows) binades,
 * and is otherwise within rows * 2^-53 relative of it.  Each row is read from
 * HBM once, whatever m is.
 *
 *   x_act     [rows, ld] fp32 or bf16 device, read only.
 *   ks        [m] HOST array, 1 <= ks[q] <= d.   m  1 .. DCT_DIAG_MAX_QUANTILES.
 *   mean_out  [m] binary64 device.
 *   tau_out   [m*rows] dtype device (required: it is also the scratch of the mean).
 * Limits and errors as dct_mp_topk_pack_fwd.
 */
DCT_API dct_status_t dct_mp_threshold_mean(
    const void* x_act, dct_dtype_t dtype, uint32_t rows, uint32_t d, uint32_t ld,
    const uint32_t* ks, uint32_t m,
    double* mean_out, void* tau_out, dct_stream_t stream);

/*
 * dct_dp_drift_check -- has the survivor count of a compress call drifted away
 * from the target k while the threshold is being reused?  (Sec. 2.1 reuses tau
 * for L iterations because it moves little around its running mean; this is the
 * guard for the case where it does move.  The paper states the observation, not
 * a monitor: the rule below is this library's.)
 *
 * Reads compress_result->needed (the true survivor count of the last
 * dct_dp_compress on this stream) and writes
 *   *flag_out = 1  if needed * ratio_den > k * ratio_num   (too dense: tau too low),
 *               2  if needed * ratio_num < k * ratio_den   (too sparse: tau too high),
 *               0  otherwise,
 * i.e. 0 while k / ratio <= needed <= k * ratio with ratio = ratio_num / ratio_den >= 1.
 * Everything stays on the device and on the stream, so a trainer can branch on the
 * flag (or capture the check in a graph) without a host round trip.
 *   compress_result  device;  flag_out  device uint32;  k >= 1;
 *   ratio_num >= ratio_den >= 1 (else DCT_ERR_INVALID_ARG).
 */
DCT_API dct_status_t dct_dp_drift_check(
    const dct_result_t* compress_result, uint64_t k,
    uint32_t ratio_num, uint32_t ratio_den,
    uint32_t* flag_out, dct_stream_t stream);

/*
 * TEST-ONLY knobs, exported for the library's own test-suite and not part of the production interface: two
 * process-wide words (atomics) that every later call reads once.  A build with -DDCT_NO_TEST_HOOKS turns the
 * call into a no-op.  spin_limit is the
 * number of polls a device-side wait may take before it gives up with
 * DCT_ERR_TIMEOUT (default 2^21, about a second).  first_ticket is the id of
 * the first tile dct_dp_compress hands out (default 0); with 1, tile 0 is never
 * processed, so its successor's bounded wait can be observed to run out without
 * wedging the GPU.  The paper has no counterpart for this call.
 */
DCT_API void dct_debug_configure(uint32_t spin_limit, uint32_t first_ticket);

#ifdef __cplusplus
}
#endif
#endif /* DCT_H_ */
