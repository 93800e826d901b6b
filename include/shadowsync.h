/*
 * shadowsync.h — C boundary of the ShadowSync hot path on one B200 (sm_100a).
 *
 * The path is the CTR training step of a DLRM-style model run by R trainer
 * replicas that live on one GPU (paper Section 3.1, Fig. 1, Algorithm 1) and
 * the paper's background synchronisation of the replicated dense parameters
 * (Algorithms 2, 3 and 4).  Every call below enqueues hand-written CUDA kernels
 * on the stream it is given and returns; nothing here runs on the CPU and there
 * is no fallback: a device that is not sm_100 gives SS_ERR_ARCH.
 *
 * General conventions
 *   - All data pointers are DEVICE pointers into caller-owned memory unless a
 *     parameter says "host".  The compute calls allocate no device memory: scratch
 *     comes from caller-provided workspaces whose sizes are queried first.
 *   - State the library keeps: the last CUDA error code of each host thread; per
 *     device, cached facts found on first use (compute capability, SM count, kernel
 *     attributes such as the dynamic shared-memory limit, driver entry points, the
 *     device addresses of its own __device__ symbols); one device-side error word
 *     (ss_device_error); the 2112 KiB built-in scratch of ss_embbag_bwd_sort_noalloc;
 *     the tuning value of ss_mlp_set_flow_ctas; while the kernel timers are on
 *     (ss_profile), pools of CUDA events and their records; and, per ss_shadow_start,
 *     a heap-allocated handle with a host thread until ss_shadow_stop.
 *     Because of the first-use set-up, make the first call of each entry point on a
 *     device outside any stream capture; later calls can be captured into CUDA graphs
 *     (the timers must be off while capturing).  Calls may come from several host
 *     threads; calls that share a workspace must be ordered by the caller.
 *   - Calls validate their arguments on the host, enqueue on `stream`
 *     (a cudaStream_t passed as void*, 0 = the legacy default stream) and
 *     return without synchronising.  Buffers must stay alive until the stream
 *     has run the work.
 *   - Return value: SS_OK or a negative ss_status.  Nothing aborts; no kernel
 *     traps.  Malformed *data* seen on the device (an index outside [0,N), a
 *     decreasing or negative offset, an offset beyond the end of the index list
 *     offsets[T*B]) ORs a bit into *d_status and that lookup or bag is skipped.
 *     A bounded wait inside a tensor-core kernel that runs out raises the device
 *     error word instead of hanging; the kernel then stores nothing more.
 *   - Row-major everywhere.  float = IEEE binary32, bf16 = bfloat16 stored as
 *     uint16_t.  "ld" = leading dimension in elements.
 *   - Pointers that are read or written with 128-bit accesses must be 16-byte
 *     aligned and their ld a multiple of 4 floats / 8 bf16 (SS_ERR_ALIGN).
 */
#ifndef SHADOWSYNC_H_
#define SHADOWSYNC_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int32_t ss_status;
enum {
  SS_OK = 0,
  SS_ERR_NULL = -1,      /* a required pointer is NULL                                   */
  SS_ERR_SHAPE = -2,     /* a size is negative, zero where it must not be, or too large  */
  SS_ERR_ALIGN = -3,     /* pointer or leading dimension not aligned for 128-bit access  */
  SS_ERR_DTYPE = -4,     /* unsupported gemm_dtype, or a bf16 buffer missing in bf16 mode */
  SS_ERR_WORKSPACE = -5, /* workspace smaller than the matching *_workspace_bytes query  */
  SS_ERR_ARCH = -6,      /* current device is not compute capability 10.x                */
  SS_ERR_CUDA = -7,      /* a CUDA call failed; see ss_last_cuda_error()                 */
  SS_ERR_RANGE = -8      /* a scalar is outside its domain (alpha not in [0,1], ...)     */
};

/* bits ORed into *d_status by kernels */
enum {
  SS_DEV_BAD_INDEX = 1,  /* a row index outside [0, N): lookup skipped                   */
  SS_DEV_BAD_OFFSET = 2, /* offsets not non-decreasing or beyond L: bag treated as empty */
  SS_DEV_BAD_WORKSPACE = 4 /* ss_embbag_bwd_apply on a workspace that holds no finished sort of this T, N, L: nothing done */
};

typedef void* ss_stream;

const char* ss_status_str(ss_status s);
int ss_last_cuda_error(void);      /* cudaError_t of the last failed CUDA call of this thread */
int ss_num_sms(void);              /* multiprocessor count of the current device, <0 on error */

/* ------------------------------------------------------------------------------------------
 * Embedding lookup + sum pooling (Section 3.1 "Embedding PS": several rows of a feature are
 * pooled next to the table and only the pooled vector goes to the trainer).
 *
 *   out[b, col0 + t*D + d] = sum_{j in [offsets[t*B+b], offsets[t*B+b+1])} tables[t, indices[j], d]
 *
 * tables   float [T, N, D]   shared by all replicas (the paper's h)
 * indices  int32 [L]         row ids, all bags of table 0 first, then table 1, ...
 * offsets  int32 [T*B + 1]   CSR bag boundaries, bag id = t*B + b, offsets[T*B] = L
 * out_f32  float [B, ld_f32] nullable; out_bf16 bf16 [B, ld_bf16] nullable; at least one given.
 *          Both are the replica's concat buffer; col0 is the first pooled column (= D when the
 *          bottom MLP output occupies columns 0..D-1).
 * D must be a multiple of 4 and at most 1024.  A row occurring twice in a bag counts twice.
 * ---------------------------------------------------------------------------------------- */
ss_status ss_embbag_fwd(const float* tables, int T, int64_t N, int D,
                        const int32_t* indices, const int32_t* offsets, int B,
                        float* out_f32, int64_t ld_f32, void* out_bf16, int64_t ld_bf16, int col0,
                        int32_t* d_status, ss_stream stream);

/* ------------------------------------------------------------------------------------------
 * Embedding backward fused with the row-wise sparse Adagrad update (Section 3.2 "Embedding
 * Tables": lock-free updates of the single table copy, optimizer state stored with the rows).
 * Deterministic: the result does not depend on thread scheduling.
 *
 *   1. key = t*N + row for each of the L lookups; stable sort by key
 *        -> perm[L] (lookup positions, ascending key, equal keys in ascending position)
 *   2. distinct keys -> uniq_keys[U]; seg_off[U+1] (segment u = perm[seg_off[u] .. seg_off[u+1]))
 *   3. g_u[d] = sum over the lookups of segment u of grad[b, col0 + t*D + d]  (b = the lookup's sample)
 *   4. s_u = row_state[key_u] + mean_d g_u[d]^2;  row_state[key_u] = s_u;
 *      tables[key_u, d] -= lr * g_u[d] / (sqrt(s_u) + eps)
 *
 * row_state float [T*N]; grad float [B, ld_grad].  uniq_keys / seg_off / perm are optional
 * outputs (NULL = keep them in the workspace only); sizes L, L+1, L.  *d_num_unique receives U.
 * T*N must be below 2^31.  The workspace holds the sort buffers; query its size first.
 * ---------------------------------------------------------------------------------------- */
size_t ss_embbag_bwd_workspace_bytes(int T, int64_t N, int D, int B, int64_t L);
ss_status ss_embbag_bwd_adagrad(float* tables, float* row_state, int T, int64_t N, int D,
                                const int32_t* indices, const int32_t* offsets, int B, int64_t L,
                                const float* grad, int64_t ld_grad, int col0, float lr, float eps,
                                void* workspace, size_t workspace_bytes,
                                int32_t* uniq_keys, int32_t* seg_off, int32_t* perm,
                                int32_t* d_num_unique, int32_t* d_status, ss_stream stream);

/* The sort half handles a table with at most this many lookups in a call with one thread block that sorts in shared
 * memory (a light kernel on T SMs); when the lookups of a call exceed T times this number, or a table exceeds it, tiled
 * passes over all SMs sort instead.  Callers that schedule the sort beside other work can plan with it. */
#define SS_TABLE_SORT_CAP 24576

/* The same operation in two calls, so that its first half can be enqueued early on another stream:
 * steps 1-2 depend only on the batch's indices, steps 3-4 also on the gradient.
 *   ss_embbag_bwd_sort   steps 1-2 into the workspace (and the optional uniq_keys / seg_off / perm outputs)
 *   ss_embbag_bwd_apply  steps 3-4 from a workspace that ss_embbag_bwd_sort filled for the same batch
 * Arguments as in ss_embbag_bwd_adagrad; the caller orders the two calls (same stream, or an event).
 * The sort stamps the workspace with (T*N, L); an apply whose T, N, L do not match the stamp changes
 * nothing and sets SS_DEV_BAD_WORKSPACE in *d_status (nullable).  A workspace sorted for another batch
 * of the same T, N, L cannot be told apart: the update is then memory-safe but meaningless. */
ss_status ss_embbag_bwd_sort(int T, int64_t N, int D, const int32_t* indices, const int32_t* offsets, int B,
                             int64_t L, void* workspace, size_t workspace_bytes,
                             int32_t* uniq_keys, int32_t* seg_off, int32_t* perm,
                             int32_t* d_num_unique, int32_t* d_status, ss_stream stream);
ss_status ss_embbag_bwd_apply(float* tables, float* row_state, int T, int64_t N, int D, int B, int64_t L,
                              const float* grad, int64_t ld_grad, int col0, float lr, float eps,
                              void* workspace, size_t workspace_bytes, int32_t* d_status, ss_stream stream);

/* The sort / unique half once more, for callers that cannot allocate.  (The paper has no counterpart:
 * this entry point exists only for how the library is embedded.)
 *
 * ss_embbag_bwd_sort needs a workspace, and whoever calls it has to get that memory from somewhere.
 * Not every caller can: a process whose allocator has already given the whole GPU to other owners, a
 * plug-in inside another program's serving loop that must not trigger cudaMalloc's device-wide
 * synchronisation, or code that runs before the application's memory pool is up.  This variant takes
 * no workspace.  Its scratch is a fixed array of 2112 KiB compiled into the library, which every GPU
 * that loads the library keeps until the process ends, so the size is capped:
 *     L <= 65536 lookups per call, otherwise SS_ERR_SHAPE (use ss_embbag_bwd_sort with a workspace).
 * It calls no cudaMalloc / cudaFree and no routine that allocates.
 *
 * Inputs as for ss_embbag_bwd_sort (no D: the sort does not depend on the row width).  Outputs, all
 * required: uniq_keys[L], seg_off[L+1], perm[L], *d_num_unique, bit-identical to ss_embbag_bwd_sort's.
 * The row update is not part of it: ss_embbag_bwd_apply wants the workspace of ss_embbag_bwd_sort.
 *
 * The first call on a device looks up the device address of the built-in array (one
 * cudaGetSymbolAddress); make that first call before any stream capture begins.  All calls, from
 * every thread and stream, share the one array: two calls that may run on the GPU at the same time
 * race and produce garbage, so put them on one stream or order them with events.  The array keeps
 * whatever the last call wrote; each call rewrites every part it reads, so no clearing is needed. */
ss_status ss_embbag_bwd_sort_noalloc(int T, int64_t N, const int32_t* indices, const int32_t* offsets, int B,
                                     int64_t L, int32_t* uniq_keys, int32_t* seg_off, int32_t* perm,
                                     int32_t* d_num_unique, int32_t* d_status, ss_stream stream);

/* ------------------------------------------------------------------------------------------
 * Bottom MLP, concat interaction, top MLP, sigmoid + binary cross-entropy (Section 3.1, Fig. 1;
 * "Trainer": forward pass, then gradients for all parameters, local parameters updated directly).
 *
 * ss_mlp_desc (host struct, host int arrays):
 *   bottom_dims[n_bottom+1]  e.g. {13, 512, 256, 64}: Linear+ReLU for every bottom layer
 *   top_dims[n_top+1]        e.g. {1728, 512, 256, 1}: Linear+ReLU, the last layer linear -> logit
 *   top_dims[0] is the concat width W; columns 0..bottom_dims[n_bottom]-1 of the concat buffer are
 *   the bottom output, the remaining columns are the pooled embeddings written by ss_embbag_fwd.
 *   gemm_dtype 0: float operands.  1: bf16 operands with float accumulation, float master weights.
 *
 * Parameter vector w^(i): ONE flat float array per replica.  Layers in order (bottom first), for
 * each layer the weight matrix [out, in] row-major, then the bias [out]; every tensor starts on a
 * multiple of 32 floats (pads are zero and stay zero under all updates).  ss_mlp_param_offsets
 * writes the start of each tensor.  The Adagrad accumulator, the optional raw-gradient output and
 * the bf16 mirror (gemm_dtype 1; mirror[k] = bf16(w[k])) share this layout.
 * ---------------------------------------------------------------------------------------- */
typedef struct {
  int n_bottom, n_top;
  const int* bottom_dims;
  const int* top_dims;
  int gemm_dtype;
} ss_mlp_desc;

int64_t ss_mlp_param_count(const ss_mlp_desc* desc);  /* padded length of the flat vector, <0 on error */
ss_status ss_mlp_param_offsets(const ss_mlp_desc* desc, int64_t* w_off, int64_t* b_off); /* host arrays [n_bottom+n_top] */
size_t ss_mlp_workspace_bytes(const ss_mlp_desc* desc, int B);

/* How the tensor-core layers run (gemm_dtype 1): all of them in ONE persistent launch per pass.  Its CTAs draw
 * 128-row output tiles of all layers from a counter in the workspace; a tile of a layer waits, inside the launch,
 * for the row blocks of the previous layer it reads (forward: activations; backward: the gradient above it; weight
 * gradients, which contract over the batch, wait k block by k block).  The workspace therefore also holds the
 * launch's control words; ss_mlp_fwd clears them, so a workspace needs no initialisation.
 *
 * Forward.  dense float [B, bottom_dims[0]]; labels float [B] in {0,1}.
 * concat_f32 [B, W] (gemm_dtype 0) / concat_bf16 [B, W] (gemm_dtype 1) must already hold the pooled
 * columns; the call fills columns 0..D0-1.  Outputs: logit[B], prob[B] = sigmoid(logit),
 * loss[1] = mean_b( max(z,0) - z*y + log(1+exp(-|z|)) ).  The workspace keeps the activations
 * that ss_mlp_bwd needs: call bwd with the same workspace before the next fwd on it. */
ss_status ss_mlp_fwd(const ss_mlp_desc* desc, const float* w, const void* w_bf16,
                     const float* dense, float* concat_f32, void* concat_bf16, int B,
                     const float* labels, float* logit, float* prob, float* loss,
                     void* workspace, size_t workspace_bytes, ss_stream stream);

/* Backward + local update.  dz = (prob - y)/B; back-propagation through top and bottom MLP.
 * grad_pooled float [B, ld_grad] receives d loss / d concat[:, D0:] (column j = concat column D0+j).
 * grads (nullable) receives the raw dW, db in the flat layout.
 * If apply_update: element-wise Adagrad on every parameter,
 *     acc += g*g;  w -= lr * g / (sqrt(acc) + eps);  w_bf16 = bf16(w)   (acc per replica, never synced). */
ss_status ss_mlp_bwd(const ss_mlp_desc* desc, float* w, void* w_bf16, float* adagrad_acc, float* grads,
                     const float* dense, const float* concat_f32, const void* concat_bf16,
                     const float* labels, const float* prob, int B, float lr, float eps, int apply_update,
                     float* grad_pooled, int64_t ld_grad,
                     void* workspace, size_t workspace_bytes, ss_stream stream);

/* ------------------------------------------------------------------------------------------
 * Normalised entropy (Section 4, "Evaluation Metrics"): the mean cross-entropy of the predictions divided
 * by the entropy of the empirical click rate.  ss_ne_accumulate adds one batch to acc (device double[3]:
 * sum of cross-entropies computed from the logits, sum of labels, count; the caller zeroes it before the
 * first batch); ss_ne_value writes NE of everything accumulated so far to out (device double[1]).
 * Fed with the logits ss_mlp_fwd returns -- predictions made before the step's update -- it gives the
 * paper's Train NE; fed with logits of held-out batches, its Eval NE.  Calls on one acc must be ordered
 * (same stream): the accumulation is a plain read-modify-write.
 * ---------------------------------------------------------------------------------------- */
ss_status ss_ne_accumulate(const float* logit, const float* labels, int B, double* acc, ss_stream stream);
ss_status ss_ne_value(const double* acc, double* out, ss_stream stream);

/* ------------------------------------------------------------------------------------------
 * Background synchronisation of the replicated dense parameters (Algorithms 2, 3, 4).  Each call
 * is ONE kernel that reads all R replica vectors and the centre/global copy once and writes them
 * back.  w: HOST array of R device pointers to float[n]; w_bf16: NULL or HOST array of R device
 * pointers to the bf16 mirrors, refreshed from the new values.  1 <= R <= 16, 0 <= alpha <= 1.
 * The kernels take no lock: run concurrently with training they race with it element by element,
 * as the paper's shadow thread does with its worker threads (Section 3.2).
 * ---------------------------------------------------------------------------------------- */
enum {
  SS_SYNC_EASGD_LITERAL = 1, /* Algorithm 2 line by line: the replica interpolates toward the updated centre */
  SS_SYNC_BMUF_NESTEROV = 2  /* Algorithm 4 with the Nesterov variant its comment allows: pull toward g + mu*delta */
};

/* Shadow EASGD (Algorithm 2), the R trainers visiting the centre in turn, r = 0..R-1:
 *   d = alpha*(w_r - c);  w_r -= d;  c += d. */
ss_status ss_sync_easgd(float* const* w, int R, float* center, int64_t n, float alpha, int flags,
                        void* const* w_bf16, ss_stream stream);

/* Shadow MA (Algorithm 3): m = (1/R) sum_r w_r;  w_r = (1-alpha) w_r + alpha m;  global_out (nullable) = m. */
ss_status ss_sync_ma(float* const* w, int R, float* global_out, int64_t n, float alpha, int flags,
                     void* const* w_bf16, ss_stream stream);

/* Shadow BMUF (Algorithm 4) with block momentum: m = mean_r w_r;  delta = mu*delta + eta*(m - g);
 *   g += delta;  w_r = (1-alpha) w_r + alpha g.   mu = 0 is the algorithm as printed.
 * flags & SS_SYNC_BMUF_NESTEROV: the replicas are pulled toward the look-ahead point g + mu*delta instead of g. */
ss_status ss_sync_bmuf(float* const* w, int R, float* global, float* delta, int64_t n,
                       float alpha, float eta, float mu, int flags,
                       void* const* w_bf16, ss_stream stream);

/* ------------------------------------------------------------------------------------------
 * The shadow thread (Section 3.2; "shadow thread do" of Algorithms 1-4): ss_shadow_start spawns a host
 * thread that loops  { one synchronisation pass on `stream` }  until ss_shadow_stop, the rule's
 * arguments as in ss_sync_easgd (rule 0), ss_sync_ma (rule 1, center = global_out) or ss_sync_bmuf
 * (rule 2).  It waits on nothing but its own earlier passes: at most max_in_flight (1..8) passes are
 * queued ahead of the device; pause_us > 0 sleeps between passes; it ends by itself after max_rounds
 * passes.  Give it a stream of the lowest priority and the training streams a higher one, and the
 * device runs the passes in whatever room training leaves.  The pointer arrays are copied; the
 * buffers they point to must outlive ss_shadow_stop, which joins the thread, waits for the queued
 * passes, stores the number of passes in *rounds_out (nullable), frees the handle and returns the
 * first error the thread met (SS_OK if none).  ss_shadow_rounds reads the running count of passes
 * enqueued.  ss_shadow_pause(h, 1) makes the thread stop enqueuing and returns once every pass it
 * had enqueued has completed on the device (ss_shadow_rounds is then the number of completed
 * passes); ss_shadow_pause(h, 0) lets it loop again.  A paused thread still ends on ss_shadow_stop.
 * ---------------------------------------------------------------------------------------- */
typedef struct ss_shadow ss_shadow;
ss_status ss_shadow_start(ss_shadow** out, int rule, float* const* w, int R, float* center, float* delta, int64_t n,
                          float alpha, float eta, float mu, int flags, void* const* w_bf16, ss_stream stream,
                          int max_in_flight, int pause_us, int64_t max_rounds);
int64_t ss_shadow_rounds(const ss_shadow* h);
ss_status ss_shadow_pause(ss_shadow* h, int paused);
ss_status ss_shadow_stop(ss_shadow* h, int64_t* rounds_out);

/* ------------------------------------------------------------------------------------------
 * The tensor-core building block of ss_mlp_fwd / ss_mlp_bwd, exposed for testing and timing:
 *   C[m, n] = sum_k A(m, k) * B(n, k),  bf16 operands, float accumulation, float C [M, ldc].
 * a_mn_major = 0: A is stored [M, lda] with k contiguous (activations, weights in the forward pass).
 * a_mn_major = 1: A is stored [K, lda] with m contiguous (the same buffers read transposed in the
 * backward pass: dW = dY^T X, dX = dY W).  Likewise for B with n.  lda, ldb multiples of 8, N a
 * multiple of 8, K >= 16, pointers 16-byte aligned, else SS_ERR_ALIGN.  force_simt = 1 runs the
 * same product on the SIMT kernel instead (any shape).
 * ss_device_error returns the device-side error flag (0 = none; k > 0 = the k-th kind of bounded
 * wait in a tensor-core kernel ran out: 1 producer, 2 MMA issuer, 3 epilogue) after synchronising
 * the device, and clears it if clear != 0.  A negative value means the flag could not be read.
 * ---------------------------------------------------------------------------------------- */
ss_status ss_gemm_bf16(const void* a, int a_mn_major, int64_t lda, const void* b, int b_mn_major, int64_t ldb,
                       float* c, int64_t ldc, int M, int N, int K, int force_simt, ss_stream stream);
int ss_device_error(int clear);

/* Tuning knob, no counterpart in the paper: how many CTAs (SMs) the persistent tensor-core launch of ss_mlp_fwd /
 * ss_mlp_bwd takes.  0 (the default) means 32, the value with which several replicas training concurrently on one device
 * got the most examples per second (CTAs of such a launch hold a whole SM's shared memory and wait for one another).
 * A pass that has the device to itself is fastest with one CTA on every SM (pass the SM count).
 * A negative value changes nothing.  Returns the number now in effect (32 while the default stands).
 * Process-wide; set it before the calls it should affect (a captured CUDA graph keeps the value it was captured with). */
int ss_mlp_set_flow_ctas(int ctas);

/* float -> bf16 (round to nearest even) of n elements; used to initialise a bf16 mirror. */
ss_status ss_to_bf16(const float* src, void* dst_bf16, int64_t n, ss_stream stream);

#ifdef __cplusplus
}
#endif
#endif /* SHADOWSYNC_H_ */
