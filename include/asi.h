/*
 * asi.h -- C ABI of the B200 (sm_100a) ASI library.
 *
 * ASI (Activation Subspace Iteration) keeps, for every trained layer, a Tucker
 * form of the layer's input activation instead of the activation itself:
 *
 *     A  ~=  S x_1 U_1 x_2 U_2 ... x_n U_n          (Sec. 3.2, Tucker form)
 *
 * with core S in R^{r_1 x .. x r_n} and factors U_m in R^{D_m x r_m} with
 * orthonormal columns.  Each training step the factors are refreshed by ONE
 * warm-started subspace iteration per mode (Algorithm 1), and the backward
 * pass computes the weight gradient from (S, U, dY) without rebuilding A
 * (appendix "Speedup", cost model C_ASI).
 *
 * Conventions common to every entry point
 *   - All tensor pointers are DEVICE pointers unless the name ends in _host.
 *   - The caller owns every buffer, including the workspace; the library
 *     allocates no device memory and keeps no mutable state in a plan, so one
 *     plan may be used from several streams (with distinct workspaces).
 *   - Tensors are contiguous, row-major: activation [B,C,H,W] (conv) or
 *     [B,N,Din] / [B,Din] (linear); dY [B,Cout,H',W'] or [..,Dout];
 *     dW [Cout, C/groups, kh, kw] or [Dout, Din]; core [r_1,..,r_n].
 *   - "U" buffers hold all factors back to back: U_m is row-major
 *     [D_m x r_m] and starts at element asi_plan_info_t.u_offset[m].
 *   - act and dY have the plan's in_dtype (fp32 or bf16); everything else is
 *     fp32.  Accumulation is fp32 or wider.
 *   - Calls are asynchronous on `stream`.  Errors the host can see are
 *     returned immediately and nothing is enqueued.  Conditions only the
 *     device can see (a rank-deficient A_m A_m^T U_m) are written to a status
 *     word at the start of the workspace and read back by asi_poll_status.
 *   - Workspaces must be 256-byte aligned.
 */
#ifndef ASI_B200_H
#define ASI_B200_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  ASI_OK = 0,
  ASI_ERR_INVALID_ARG = 1,    /* null pointer, bad enum, non-positive size, aliasing */
  ASI_ERR_UNSUPPORTED = 2,    /* dilation != 1, rank > 128, ndim out of range */
  ASI_ERR_RANK_RANGE = 3,     /* r_m outside [1, min(a_m, b_m)] (Algorithm 1, inputs) */
  ASI_ERR_WORKSPACE = 4,      /* workspace too small or misaligned */
  ASI_ERR_CUDA = 5,           /* a CUDA runtime call failed */
  ASI_ERR_RANK_DEFICIENT = 6, /* device: Orthogonalize met a dependent column */
  ASI_ERR_TIMEOUT = 7         /* device: a bounded wait expired */
} asi_status_t;

typedef enum { ASI_F32 = 0, ASI_BF16 = 1 } asi_dtype_t;
typedef enum { ASI_CONV2D = 0, ASI_LINEAR = 1 } asi_kind_t;

#define ASI_MAX_MODES 4
#define ASI_MAX_RANK 128

/* One trained layer.  conv: ndim = 4, dims = (B,C,H,W).  linear: ndim = 2 or 3,
 * dims = (B[,N],Din), cout = Dout and the conv fields are ignored. */
typedef struct {
  int32_t kind;                  /* asi_kind_t */
  int32_t in_dtype;              /* asi_dtype_t of act and dY */
  int32_t ndim;
  int64_t dims[ASI_MAX_MODES];
  int32_t ranks[ASI_MAX_MODES];  /* 1 <= r_m <= min(a_m, b_m), r_m <= ASI_MAX_RANK */
  int32_t cout;
  int32_t kh, kw, stride_h, stride_w, pad_h, pad_w, dil_h, dil_w, groups;
  int32_t flags;                 /* ASI_FLAG_* bits, 0 for defaults */
} asi_layer_desc_t;

/* Use only the shape-generic kernels even where a fused kernel covers the layer
 * (same results up to fp32 rounding; for testing and comparison). */
#define ASI_FLAG_GENERIC_ONLY 1
/* Test hook for the bounded device waits: on the fused small-map path the producer of the bulk copy arms
 * its barrier but issues no copy, and the wait limit drops from one second to one millisecond, so the
 * waiting CTAs run into the limit, record ASI_ERR_TIMEOUT in the status word and return.  The outputs
 * of such a call are undefined; nothing faults and the workspace can be used again afterwards. */
#define ASI_FLAG_TEST_EXPIRE_WAIT 2
/* The layer's kernels are expected to run beside kernels of other layers (one CUDA-graph branch or one stream
 * per layer; Algorithm 1 treats every fine-tuned layer of a step independently).  The streaming kernels of
 * large feature maps then launch one CTA per SM instead of two, which leaves registers and shared memory for
 * the neighbours: alone they run about 5 % slower, ten layers side by side about 4 % faster.  Results are the
 * same up to the order of the per-CTA partial sums (a fixed order per plan). */
#define ASI_FLAG_SHARE_SM 4

/* Sizes and the paper's closed forms for one plan. */
typedef struct {
  size_t compress_ws_bytes;      /* workspace asi_compress needs */
  size_t wgrad_ws_bytes;         /* workspace asi_*_wgrad needs */
  int64_t u_offset[ASI_MAX_MODES];
  int64_t u_elems;               /* sum_m D_m r_m */
  int64_t core_elems;            /* prod_m r_m */
  int64_t act_elems, dy_elems, dw_elems;
  int64_t out_h, out_w;          /* conv output size H', W' */
  int64_t compressed_elems;      /* M_i = prod r_m + sum D_m r_m   (Sec. 3.2, storage equation) */
  double ratio_RC;               /* prod D_m / M_i                  (appendix, space complexity) */
  double macs_O_ASI;             /* sum_m (2 a_m b_m r_m + r_m^3)   (appendix, overhead) */
  double macs_C_ASI;             /* five-term backward cost         (appendix, speedup); conv only, else 0 */
  double macs_C_vanilla;         /* D^2 C C' B H' W' (conv) or B N Din Dout (linear) */
} asi_plan_info_t;

typedef struct asi_plan asi_plan_t;

/* Host only; validates the descriptor and fixes kernel variants and workspace
 * layout.  No GPU work, no CUDA context needed.  *out is set only on ASI_OK. */
asi_status_t asi_plan_create(const asi_layer_desc_t* desc, asi_plan_t** out);
asi_status_t asi_plan_destroy(asi_plan_t* plan);
asi_status_t asi_plan_query(const asi_plan_t* plan, asi_plan_info_t* info);

/* Algorithm 1 (ASI), branch t > 0, for one layer and one step:
 *   for every mode m (each on the ORIGINAL activation):
 *       V = A_m^T U_m^{prev};  U_m^{new} = Orthogonalize(A_m V)
 *   core = A x_1 U_1^{new T} ... x_n U_n^{new T}
 * Orthogonalize returns the Gram-Schmidt basis (thin-QR Q with diag(R) > 0).
 *   act     [in]  device, in_dtype, dims as planned; not modified
 *   U_prev  [in]  device fp32, u_elems; previous step's factors
 *   U_new   [out] device fp32, u_elems; must not alias U_prev
 *   core    [out] device fp32, core_elems
 *   ws      device scratch of at least compress_ws_bytes; contents undefined
 *           afterwards except the status word.
 * All work is ordered after what `stream` held before the call and before what is enqueued on it
 * afterwards.  For 3-mode linear layers the passes of the modes run side by side on two streams owned
 * by the plan (created at the plan's first call on the current device; the plan keeps using that
 * device's streams), forked from and joined to `stream` by events, so the call may be captured into a
 * CUDA graph like any other. */
asi_status_t asi_compress(const asi_plan_t* plan, const void* act, const float* U_prev,
                          float* U_new, float* core, void* ws, size_t ws_bytes, void* stream);

/* Algorithm 1, branch t = 0 (cold start) with caller-supplied Gaussian test
 * matrices: U_m = Orthogonalize(A_m Omega_m), then the core as above.
 *   omega  [in] device fp32: Omega_m row-major [b_m x r_m], modes back to back
 *          (offset of mode m = sum_{j<m} b_j r_j), rows ordered like the
 *          columns of the mode-m unfolding with the remaining modes in
 *          increasing order, last mode fastest. */
asi_status_t asi_init_factors(const asi_plan_t* plan, const void* act, const float* omega,
                              float* U_new, float* core, void* ws, size_t ws_bytes, void* stream);

/* The same cold start with the Gaussian test matrices drawn by the library (Algorithm 1, t = 0: "V ~ N(0, 1)";
 * the paper names no generator).  Omega_m is the first b_m r_m values of the counter-based stream
 * (seed, stream = m): Philox4x32-10 with key = seed and counter = (group index, stream, 0), a word x mapped to
 * u = ((x >> 9) + 0.5) 2^-23, pairs of words through Box-Muller in fp32; element e of a stream is value e mod 4
 * of group e div 4.  The matrices are drawn mode by mode into the workspace, so the caller holds no Omega and
 * the scratch grows by the largest b_m r_m floats only.  Same seed, same plan: same factors.
 *   ws  device scratch of at least asi_init_seeded_ws_bytes(plan). */
size_t asi_init_seeded_ws_bytes(const asi_plan_t* plan);
asi_status_t asi_init_factors_seeded(const asi_plan_t* plan, const void* act, uint64_t seed, float* U_new,
                                     float* core, void* ws, size_t ws_bytes, void* stream);
/* The generator by itself: out[0..n) = the first n values of the N(0, 1) stream (seed, stream_id) (device fp32),
 * and the raw words of its first n_groups groups (device uint32, 4 per group, 16-byte aligned). */
asi_status_t asi_gaussian_stream(uint64_t seed, uint32_t stream_id, int64_t n, float* out, void* stream);
asi_status_t asi_philox_words(uint64_t seed, uint32_t stream_id, int64_t n_groups, uint32_t* out, void* stream);

/* The layers one training step handles together, in one call each way: Algorithm 1 is run for every
 * fine-tuned layer at every step (Sec. 4 fine-tunes the last two to four layers), and the backward pass
 * needs every layer's weight gradient.  Arrays of n entries, entry i as in asi_compress / asi_*_wgrad;
 * every layer has its own workspace (distinct pointers).  Results are bit-identical to n separate
 * calls.  Layers on the fused small-map path that share a kernel variant (map size, rank bucket, input
 * type) share one launch per kernel stage -- a step of L such layers is 3 + 1 launches instead of
 * 3L + L --, the others are enqueued one after another on `stream`.  Host-detectable errors are checked
 * for all layers before anything is enqueued. */
asi_status_t asi_compress_batched(const asi_plan_t* const* plans, const void* const* acts,
                                  const float* const* U_prev, float* const* U_new, float* const* cores,
                                  void* const* ws, const size_t* ws_bytes, int32_t n, void* stream);
asi_status_t asi_wgrad_batched(const asi_plan_t* const* plans, const float* const* cores,
                               const float* const* U, const void* const* dY, float* const* dW,
                               void* const* ws, const size_t* ws_bytes, int32_t n, void* stream);

/* asi_compress for callers that cannot allocate device memory.  (The paper has no counterpart:
 * this is a deployment convenience, not part of the method.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- a training-loop hook that must
 * not disturb the framework's caching allocator, a latency-critical loop in which an allocation
 * (which synchronises the device) is not acceptable, or a process whose device-memory budget was
 * fixed at start-up.  Such a caller still owns act, U_prev, U_new and core, but has nowhere to
 * get the scratch workspace from.
 *
 * This entry point computes exactly what asi_compress computes, with the workspace taken from an
 * array of ASI_STATIC_WS_MAX_BYTES that is part of the library image: every GPU that loads the
 * library holds that array until the process exits.  It calls no cudaMalloc / cudaFree and no
 * allocating library routine.
 *   - A plan whose compress_ws_bytes exceeds ASI_STATIC_WS_MAX_BYTES is refused with
 *     ASI_ERR_WORKSPACE and nothing is enqueued (asi_last_cuda_error() then holds the two sizes).
 *   - The first call on each device looks up the array's device address (one runtime query, with
 *     that device current).  Make that first call before any stream capture begins.  The address is
 *     remembered per device: after cudaDeviceReset it is stale, so do not reset a device between calls.
 *   - All calls on one device share the one array, and it keeps whatever the previous call left in
 *     it.  The words that must start at zero (status word, completion counters) are cleared by the
 *     call itself.  Two calls whose GPU work overlaps -- different streams, or several host threads
 *     -- race on the array: keep them on one stream or order them with events.
 *   - The device status word sits inside the shared array, so asi_poll_status cannot be used with
 *     this variant: a rank-deficient iterate is not reported.  Use asi_compress with a workspace
 *     of your own when you need that check. */
#define ASI_STATIC_WS_MAX_BYTES (4u << 20)
asi_status_t asi_compress_static_ws(const asi_plan_t* plan, const void* act, const float* U_prev,
                                    float* U_new, float* core, void* stream);

/* Weight gradient of a conv2d layer from the compressed activation, in the
 * order the five terms of C_ASI fix (appendix "Speedup"):
 *   Z1 = dY x_1 U_1^T;  Z3 = core x_3 U_3 x_4 U_4;
 *   Z4 = conv_wgrad(Z3, Z1) with the layer's kernel/stride/padding;
 *   dW = Z4 x_2 U_2  (per group when groups > 1).
 * Equals the vanilla gradient (Sec. 3.1) of the reconstructed activation.
 *   core, U [in] device fp32 (outputs of asi_compress);  dY [in] device in_dtype
 *   dW [out] device fp32 [Cout, C/groups, kh, kw], overwritten. */
asi_status_t asi_conv_wgrad(const asi_plan_t* plan, const float* core, const float* U,
                            const void* dY, float* dW, void* ws, size_t ws_bytes, void* stream);

/* Same for a linear layer y = x W^T on [B(,N),Din] tokens:
 *   Z = dY x_1 U_1^T (x_2 U_2^T);  Z4[o,k] = sum Z[..,o] core[..,k];  dW = Z4 U_last^T.
 *   dW [out] device fp32 [Dout, Din]. */
asi_status_t asi_linear_wgrad(const asi_plan_t* plan, const float* core, const float* U,
                              const void* dY, float* dW, void* ws, size_t ws_bytes, void* stream);

/* Rank selection aids (run once per layer before training, not per step).
 *
 * asi_mode_spectrum: for every mode m the leading eigenvalues of A_m A_m^T -- the squared singular values
 * of the mode-m unfolding, whose partial sums are the "explained variance" HOSVD_eps truncates by
 * (Sec. 3.2) -- in descending order, and the mode's total energy trace(A_m A_m^T) = ||A||_F^2.
 *   eig     [out] device fp64 [ndim][ASI_SPECTRUM_MAX], zero-padded; for a_m <= ASI_SPECTRUM_MAX the whole
 *           spectrum (Jacobi), otherwise the ASI_SPECTRUM_MAX leading Ritz values of a block subspace
 *           iteration on A_m A_m^T (the leading ones converged to fp64 accuracy, the trailing ones lower
 *           bounds)
 *   energy  [out] device fp64 [ndim]
 *   ws      device scratch of at least asi_spectrum_ws_bytes(plan), 256-byte aligned
 * asi_pick_ranks: the HOSVD_eps rule on those numbers: r_m = the smallest r whose leading eigenvalues
 * hold a fraction >= eps of the mode's energy, clipped to [1, min(r_max, a_m, b_m)] (Algorithm 1, rank
 * range);  ranks [out] device int32 [ndim].
 * asi_perplexity: the activation perplexity of Sec. 3.3 for one layer, ||dW - dW_approx||_F over n fp32
 * values;  out [out] device fp64 [1];  ws of at least asi_perplexity_ws_bytes(). */
#define ASI_SPECTRUM_MAX 128
size_t asi_spectrum_ws_bytes(const asi_plan_t* plan);
asi_status_t asi_mode_spectrum(const asi_plan_t* plan, const void* act, double* eig, double* energy, void* ws,
                               size_t ws_bytes, void* stream);
asi_status_t asi_pick_ranks(const asi_plan_t* plan, const double* eig, const double* energy, double eps,
                            int32_t r_max, int32_t* ranks, void* stream);
size_t asi_perplexity_ws_bytes(void);
asi_status_t asi_perplexity(const float* dW, const float* dW_approx, int64_t n, double* out, void* ws,
                            size_t ws_bytes, void* stream);

/* One whole layer-step from HOST buffers (pinned memory recommended): copies
 * act, dY and U_prev to the caller's device arena, runs asi_compress and the
 * matching wgrad, and copies U_new, core and dW back.  Everything is enqueued
 * on `stream`; the host buffers may be read after the stream is synchronised.
 *   arena  device scratch of at least asi_step_host_arena_bytes(plan). */
size_t asi_step_host_arena_bytes(const asi_plan_t* plan);
asi_status_t asi_step_host(const asi_plan_t* plan, const void* act_host, const void* dY_host,
                           const float* U_prev_host, float* U_new_host, float* core_host,
                           float* dW_host, void* arena, size_t arena_bytes, void* stream);

/* The device status of the last asi_step_host call on `arena` (its workspace sits inside the arena at
 * an offset only the library knows).  Synchronises `stream`. */
asi_status_t asi_step_host_status(const asi_plan_t* plan, const void* arena, void* stream,
                                  asi_status_t* device_status);

/* Reads the device status word of a workspace after synchronising `stream`.
 * *device_status is ASI_OK, ASI_ERR_RANK_DEFICIENT or ASI_ERR_TIMEOUT. */
asi_status_t asi_poll_status(const asi_plan_t* plan, const void* ws, void* stream,
                             asi_status_t* device_status);

/* Number of kernel launches the last call of each kind enqueues for this plan. */
int32_t asi_launch_count(const asi_plan_t* plan, int32_t which /* 0 compress, 1 wgrad */);

/* Timing aid for benchmarks: while active, every launch of kernel family `kernel_id` is
 * bracketed by cudaEventRecord on its own stream, using the caller's events pairwise:
 * events[2i] before and events[2i+1] after the i-th such launch (launches beyond n_pairs are
 * counted but not recorded).  Process-global and not thread-safe: enable it from one thread,
 * for one measurement pass, never during stream capture.  asi_profile_end returns the number
 * of launches seen since asi_profile_begin, stores in *alg_bytes (if not null) the sum over
 * those launches of the bytes each launch must move at least -- its distinct inputs read once
 * plus its outputs written once -- and switches recording off. */
typedef enum {
  ASI_K_MODEPROD = 1,     /* small-mode contraction (projection, core products, Z1, Z3, expansions) */
  ASI_K_EXPAND = 2,       /* P_m = A_m V_m */
  ASI_K_QR = 3,           /* Orthogonalize */
  ASI_K_CONV_TAIL = 4,    /* terms 4-5 of the backward cost: Z4 and dW */
  ASI_K_SM_PASS1 = 5,     /* small-map conv: all four P_m in one pass over the activation */
  ASI_K_SM_CORE = 6,      /* small-map conv: core tensor */
  ASI_K_SM_WGRAD = 7      /* small-map conv: whole compressed weight gradient */
} asi_kernel_id_t;
asi_status_t asi_profile_begin(int32_t kernel_id, void** events, int32_t n_pairs);
int32_t asi_profile_end(double* alg_bytes);

const char* asi_status_string(asi_status_t s);

/* Text of the CUDA runtime error behind the most recent ASI_ERR_CUDA on this thread
 * ("" if none).  The pointer stays valid until the next failing call. */
const char* asi_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* ASI_B200_H */
