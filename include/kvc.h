/*
 * kvc.h -- C ABI of the KVCapsule decode-time hot path for NVIDIA B200 (sm_100a).
 *
 * KVCapsule (arxiv 2605.16439) keeps a VLM backbone unchanged and stores, per layer, the
 * vision-token K/V of each n-token image block in compressed form ("capsules"):
 *   keys   : the m = ceil(l_r n) rows picked by a fixed index set M_l          (Sec. 3.1, keys)
 *   values : V_tilde = U_l (V - 1 mu_l^T), a projection along the token axis  (Sec. 3.1, values)
 * and, at every decode step, attends over the reconstructed vision K/V together with the
 * untouched text K/V (Sec. 3.2).  The library never writes full-size vision K/V: it follows
 * the associative order of Algorithm 1 (scores in compressed space, expansion by theta,
 * softmax, re-projection by U^T, product with V_tilde plus the mu term).
 *
 * Conventions
 *   - Every tensor pointer is a DEVICE pointer to caller-owned, contiguous memory unless a
 *     comment says "host".  The library owns only the opaque kvc_layer (a host struct plus a
 *     small device copy of the index set).
 *   - Calls are asynchronous on the given CUDA stream (a cudaStream_t passed as void*; NULL is
 *     the legacy default stream).  They never synchronise and, except kvc_layer_create /
 *     kvc_layer_destroy, never allocate or free device memory.
 *   - All functions returning int return a kvc_status.  Argument and shape errors are found on
 *     the host before anything is launched.  No exception crosses this boundary.
 *   - Layouts are row-major with the last index fastest; d (head dimension) must be 128.
 *   - dtype is the storage type of q, K, V, capsules, theta, U, mu and out; all arithmetic
 *     accumulates in fp32.
 */
#ifndef KVC_H_
#define KVC_H_

#include <stddef.h>
#include <stdint.h>

#if defined(KVC_BUILD) && defined(__GNUC__)
#define KVC_API __attribute__((visibility("default")))
#else
#define KVC_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  KVC_OK = 0,
  KVC_ERR_ARG = -1,        /* null pointer, negative size                               */
  KVC_ERR_SHAPE = -2,      /* unsupported or inconsistent shape                         */
  KVC_ERR_DTYPE = -3,      /* unknown dtype                                             */
  KVC_ERR_NO_PARAMS = -4,  /* theta / U / mu / idx missing for a ratio > 0              */
  KVC_ERR_WORKSPACE = -5,  /* workspace pointer null or misaligned                      */
  KVC_ERR_CUDA = -6,       /* a CUDA runtime call failed (launch, copy, allocation)     */
  KVC_ERR_TIMEOUT = -7,    /* a bounded device-side wait gave up                        */
  KVC_ERR_BOUNDS = -8      /* an index set entry is out of range or not increasing      */
} kvc_status;

typedef enum { KVC_F32 = 0, KVC_BF16 = 1 } kvc_dtype;

/* Which sides of the cache are compressed.  KVC_MODE_KV is the method (Sec. 3.1).  The one-sided settings of the
 * ablation on K-side and V-side reconstruction (App. G, Table 6) keep the other side verbatim:
 *   KVC_MODE_K_ONLY  K_tilde = the m retained key rows (theta expands the scores), V stored with all n rows per block:
 *                    out = softmax(sigma q [theta^T K_tilde ; K_txt]^T) [V ; V_txt]          (no U, no mu)
 *   KVC_MODE_V_ONLY  K stored with all n rows per block, V_tilde = U (V - 1 mu^T):
 *                    out = softmax(sigma q [K ; K_txt]^T) [U^T V_tilde + 1 mu^T ; V_txt]     (no idx, no theta) */
typedef enum { KVC_MODE_KV = 0, KVC_MODE_K_ONLY = 1, KVC_MODE_V_ONLY = 2 } kvc_mode;

/* One parameter set = one (layer, compression ratio); the paper trains M_l, theta_l, U_l, mu_l
 * per layer for a given retention ratio (App. C, Algorithm 2) and fixes them at inference
 * (Sec. 3.2).  Shapes follow App. D: theta, U in R^{H_kv x m x n}, mu in R^{H_kv x d}. */
typedef struct {
  int layer;              /* informational                                                    */
  int H_q, H_kv;          /* query heads, KV heads; G = H_q / H_kv must be an integer <= 16    */
  int d;                  /* head dimension, must be 128                                       */
  int n;                  /* tokens per vision block ("an image with size n", Sec. 3.1)        */
  int ratio_permille;     /* compression ratio rho * 1000 in [0, 1000); l_r = 1 - rho          */
  int dtype;              /* kvc_dtype                                                         */
  const int32_t* idx;     /* HOST pointer: retained-key indices, 0-based, strictly increasing; */
  int idx_per_head;       /*   [m] if 0, [H_kv][m] if 1.  Ignored when ratio_permille == 0.    */
  const void* theta;      /* [H_kv][m][n]  key / score reconstruction matrix (borrowed)        */
  const void* U;          /* [H_kv][m][n]  value PCA basis (borrowed); rows need not be orthonormal */
  const void* mu;         /* [H_kv][d]     value centering vector (borrowed)                   */
  int mode;               /* kvc_mode; 0 = both sides compressed.  K_ONLY ignores U and mu,    */
                          /*   V_ONLY ignores idx and theta (they may be NULL)                 */
} kvc_layer_desc;

typedef struct kvc_layer kvc_layer;

/* m = ceil((1 - rho) n) (Sec. 3.1), computed as (n*(1000-ratio_permille)+999)/1000 in integers.
 * Returns -1 for n <= 0 or a ratio outside [0, 1000). */
KVC_API int kvc_retained_len(int n, int ratio_permille);

/* Validates the descriptor (KVC_ERR_SHAPE / _DTYPE / _NO_PARAMS / _BOUNDS), copies the index set
 * to device memory and returns a handle.  theta, U and mu are borrowed: they must stay valid and
 * unchanged while the handle is in use.  ratio_permille == 0 is the pass-through limit: m = n,
 * capsules hold K and V verbatim, idx / theta / U / mu are ignored.
 * The device that is current at this call must be current for every later call with the handle.
 * bf16 decode calls run Alg. 1 either as one kernel (steps 2-3 on mma.sync with the logits in registers, or on tcgen05
 * with the logits in tensor memory) or, for block lengths above 640, as three kernels (streaming scores, tcgen05
 * expansion per 128 rows and range of the n axis, streaming output); the library picks per shape (same results within
 * the bf16 tolerance).  The environment variable KVC_EXPANSION = "tcgen05" | "mma" | "pair" | "split" | "resident", read when the
 * handle is created, forces one of them where it applies ("pair": the tcgen05 one-kernel path run by clusters of two
 * CTAs per (sequence, KV head)); "phases" forces the generic three-phase kernels that also serve fp32 storage. */
KVC_API int kvc_layer_create(const kvc_layer_desc* desc, kvc_layer** out);
KVC_API int kvc_layer_destroy(kvc_layer* layer);
/* Tells the handle that a capsule store it is used with has been written by something other than kvc_compress*: the next
 * decode call on the handle reads the store only after the stream's previous kernel has finished (see kvc_decode_attend). */
KVC_API int kvc_layer_capsules_written(kvc_layer* layer);

/* Bytes of the capsule store for B sequences of R blocks:  K_tilde [B][H_kv][R][m_k][d] followed
 * by V_tilde [B][H_kv][R][m_v][d] (the compressed-cache term of App. D, Eq. 2, vision part), with m_k = m_v = m
 * unless a one-sided mode keeps a side verbatim (then n rows per block on that side). */
KVC_API size_t kvc_capsule_bytes(const kvc_layer* layer, int B, int R);

/* Rows per block the capsule store holds on the key side (m_k) and on the value side (m_v); either pointer may be
 * NULL.  KVC_ERR_ARG for a NULL handle. */
KVC_API int kvc_layer_rows(const kvc_layer* layer, int* key_rows, int* value_rows);

/* Bytes of scratch kvc_decode_attend needs for B sequences of R blocks and up to T_cap text rows
 * (the figure grows with T_cap but is not monotone in B and R: size it for the B and R you call
 * with).  The scratch holds only temporaries of one call (compressed scores, expanded-probability
 * projections, split partials); it needs no initialisation and must be 256-byte aligned. */
KVC_API size_t kvc_workspace_bytes(const kvc_layer* layer, int B, int R, int T_cap);

/* Prefill-stage compression (Sec. 3.2 "Prefilling Stage").  For every sequence b, KV head h and
 * block r:  K_tilde[b,h,r,j,:] = K_vis[b,h,r*n + idx[j],:],
 *           V_tilde[b,h,r]     = U[h] (V_vis[b,h,r*n:(r+1)*n] - 1 mu[h]^T).
 * K_vis, V_vis: [B][H_kv][R*n][d].  capsules: out, kvc_capsule_bytes(layer,B,R) bytes.
 * B == 0 or R == 0 is a no-op. */
KVC_API int kvc_compress(const kvc_layer* layer, const void* K_vis, const void* V_vis, int B, int R,
                 void* capsules, void* stream);

/* Decode-stage attention over reconstructed vision K/V plus text K/V (Sec. 3.2 "Decoding Stage",
 * Algorithm 1).  out[b,hq,:] = softmax_over(R*n + T)( sigma q . [theta^T K_tilde ; K_txt] ) .
 * [U^T V_tilde + 1 mu^T ; V_txt],  sigma = 1/sqrt(d), query head hq reading KV head hq / G.
 * q, out: [B][H_q][d].  K_txt, V_txt: [B][H_kv][T_cap][d] of which the first T rows are valid
 * (may be NULL when T == 0).  R == 0 attends over text only; R == 0 and T == 0 is KVC_ERR_SHAPE.
 * workspace: kvc_workspace_bytes(layer, B, R, T_max) bytes for the same B and R and any
 * T_max >= T; calls sharing a workspace must be stream-ordered.  All per-call device state (partials, arrival
 * words, status word) lives in the workspace, none in the layer handle: calls on one handle with different
 * workspaces may run concurrently on different streams.
 * Early reads: the capsule store and the layer's parameters are fixed once written (Sec. 3.2: masks, reconstructors,
 * bases and centring vectors are fixed at inference; the compressed cache is written at prefill).  A decode call may
 * therefore begin to read them while the kernel that precedes it in the stream is still running; q, K_txt, V_txt, out
 * and the workspace are touched only after that kernel has finished.  The first decode call on a handle after a
 * kvc_compress / kvc_compress_ragged call on that handle reads the store late as well.  If anything else writes into a
 * capsule store (a kernel of the caller that swaps cache pages in, say), call kvc_layer_capsules_written(layer) before
 * the next decode call on it (copies issued with cudaMemcpyAsync need nothing: a kernel never overtakes a copy). */
KVC_API int kvc_decode_attend(const kvc_layer* layer, const void* q, const void* capsules, int B, int R,
                      const void* K_txt, const void* V_txt, int T, int T_cap, void* out,
                      void* workspace, void* stream);

/* Batches with per-sequence lengths (App. D, Eqs. 1-2 count c, n and t per request; Sec. 3.2 "Prefilling Stage"
 * compresses each request's own vision tokens).
 *
 * kvc_compress_ragged: K_vis, V_vis [B][H_kv][N_cap][d], sequence b using its first N_v[b] rows (N_v: DEVICE int[B]).
 * The floor(N_v[b] / n) whole blocks of a sequence are compressed into blocks [0, R_b[b]) of a capsule store laid out
 * for R_max blocks per sequence (kvc_capsule_bytes(layer, B, R_max) bytes; blocks a sequence does not have are left
 * untouched).  The paper compresses whole n-token blocks and is silent about a vision run that is not a whole number
 * of them: here the N_v[b] mod n rows left over stay uncompressed and are copied to rows [0, T_b[b]) of K_tail, V_tail
 * [B][H_kv][T_cap][d], the caller's text buffers, in front of which they are attended like text rows; the caller
 * appends the text rows behind them and adds their count to T_b.  R_b, T_b: DEVICE int[B], written by the call.
 * A length that does not fit (N_v[b] outside [0, N_cap], more than R_max blocks, more than T_cap rows left over) is
 * clamped and reported as KVC_ERR_BOUNDS by kvc_read_compress_status.
 *
 * kvc_decode_attend_ragged: kvc_decode_attend where sequence b attends to its first R_b[b] <= R_max blocks and its
 * first T_b[b] <= T_max <= T_cap text rows (DEVICE int[B] arrays read by the kernels, so the call can be replayed
 * with new lengths; a NULL array means R_max, or T_max, for every sequence).  T_max is an upper bound of T_b the caller
 * knows (T_cap if nothing better).  A sequence with R_b[b] == 0 and T_b[b] == 0 gets a zero output row.  Lengths
 * outside their range are clamped and reported as KVC_ERR_BOUNDS by kvc_read_device_status(layer, B, R_max, T_max, ..).
 * workspace: kvc_workspace_bytes(layer, B, R_max, T_cap).  Every sequence's result equals the call made for that
 * sequence alone. */
KVC_API int kvc_compress_ragged(const kvc_layer* layer, const void* K_vis, const void* V_vis, int B, int N_cap,
                        const int* N_v, int R_max, void* capsules, void* K_tail, void* V_tail, int T_cap,
                        int* R_b, int* T_b, void* stream);
KVC_API int kvc_decode_attend_ragged(const kvc_layer* layer, const void* q, const void* capsules, int B, int R_max,
                             const int* R_b, const void* K_txt, const void* V_txt, int T_max, const int* T_b,
                             int T_cap, void* out, void* workspace, void* stream);

/* Parameter fits from activations (App. C, Algorithm 2), on the device in fp64.  Calibration-time calls: each one
 * SYNCHRONISES the stream several times (the eigen-solver checks convergence on the host) and returns with its outputs
 * complete.  X_vis: [B][H_kv][R*n][d] device, storage type `dtype`; every n-row block of every sequence is one sample.
 * workspace: kvc_fit_workspace_bytes(H_kv, n) bytes, 256-byte aligned, device.  sweeps_out (may be NULL): sweeps the
 * eigen-solver took.  Errors: KVC_ERR_ARG / _SHAPE (m outside [1, n]) / _DTYPE / _WORKSPACE / _BOUNDS (index set) / _CUDA.
 *
 * kvc_fit_value_pca: FitValuePCA (Sec. 3.1 "Sequence-Level Low-Rank Compression for Values"): mu_out [H_kv][d] = the
 * mean of the value rows over samples and positions; U_out [H_kv][m][n] = the top-m principal directions along the
 * token axis of the centred values (eigenvectors of the n x n token covariance by a hand-written cyclic Jacobi solver;
 * rows orthonormal, each with its entry of largest magnitude positive), both written in `dtype`.  eig_out (may be
 * NULL): DEVICE double [H_kv][n], the covariance eigenvalues in descending order (squared singular values of the
 * pooled centred columns; the energy the projection loses is the sum of entries m..n-1).
 *
 * kvc_fit_key_reconstructor: for the fixed retained index set idx (HOST, as in kvc_layer_desc), theta_out [H_kv][m][n]
 * minimising sum over samples of || K - theta^T K[idx] ||_F^2, the reconstruction term of Algorithm 2 for a reconstructor
 * that is linear along the token axis; minimum-norm solution: eigen-directions of the retained rows' second-moment
 * matrix with eigenvalue <= rcond * the largest are dropped. */
KVC_API size_t kvc_fit_workspace_bytes(int H_kv, int n);
KVC_API int kvc_fit_value_pca(const void* V_vis, int B, int R, int H_kv, int n, int m, kvc_dtype dtype, void* U_out,
                      void* mu_out, double* eig_out, void* workspace, void* stream, int* sweeps_out);
KVC_API int kvc_fit_key_reconstructor(const void* K_vis, int B, int R, int H_kv, int n, int m, const int32_t* idx,
                              int idx_per_head, double rcond, kvc_dtype dtype, void* theta_out, void* workspace,
                              void* stream, int* sweeps_out);

/* Uncompressed decode attention over K, V [B][H_kv][S_cap][d] (first S rows valid), the standard
 * attention of Sec. 3.1; the comparator the compressed path is measured against.  Uses the same
 * workspace rule with R = 0, T_cap = S_cap. */
KVC_API int kvc_attend_full(const kvc_layer* layer, const void* q, const void* K, const void* V, int B,
                    int S, int S_cap, void* out, void* workspace, void* stream);

/* Decode attention without a caller-provided scratch buffer (an addition of this library; the
 * paper has no counterpart).  Same arguments, result and errors as kvc_decode_attend, minus the
 * workspace: the temporaries go to a fixed KVC_STATIC_SCRATCH_BYTES array inside the library's
 * device image, so the call performs no device allocation of any kind.  It is meant for callers
 * that cannot allocate where they decode: an engine whose memory pool is fully committed to KV
 * blocks, code running under an allocator it does not own, or a loop in which an allocation's
 * implicit device synchronisation is unacceptable.
 *   - Limit: the shape must need at most KVC_STATIC_SCRATCH_BYTES of scratch (what
 *     kvc_workspace_bytes(layer, B, R, T) reports); larger shapes return KVC_ERR_WORKSPACE
 *     ("workspace ...: static scratch too small") and nothing is launched.
 *   - The array costs KVC_STATIC_SCRATCH_BYTES of device memory on every GPU that loads the
 *     library, for the life of the process.
 *   - The first call on each device looks up the array's device address (with that device
 *     current); make that first call outside any stream capture.
 *   - All calls on a device share the one array and it keeps the previous call's contents.  The
 *     kernels clear the few words that must start at zero themselves, so no reset is needed,
 *     but two calls whose kernels overlap on the GPU (different streams, no ordering) race on it:
 *     order them on one stream or with events. */
#define KVC_STATIC_SCRATCH_BYTES (16u << 20)
KVC_API size_t kvc_static_scratch_bytes(void);
KVC_API int kvc_decode_attend_static(const kvc_layer* layer, const void* q, const void* capsules, int B,
                                     int R, const void* K_txt, const void* V_txt, int T, int T_cap,
                                     void* out, void* stream);

/* Device status word of the last kvc_decode_attend call that used `workspace` with these B, R, T:
 * 0, or KVC_ERR_TIMEOUT if a bounded device-side wait (bulk-copy completion) gave up, in which case
 * that call's output is invalid.  workspace == NULL reads the word of the last kvc_decode_attend_static
 * call on the current device.  Synchronous (copies one int to the host); the kernels never trap
 * or spin without limit. */
KVC_API int kvc_read_device_status(const kvc_layer* layer, int B, int R, int T, const void* workspace,
                                   int* status_out);

/* Device status word of the last kvc_compress call on this handle (cleared when a compress call starts):
 * 0, or KVC_ERR_TIMEOUT if a bounded wait of the value-projection kernel gave up, in which case the capsules
 * of that call are invalid.  Synchronous; call it after the stream of that kvc_compress has been synchronised.
 * Compress calls on one handle must be stream-ordered (they share this word and nothing else). */
KVC_API int kvc_read_compress_status(const kvc_layer* layer, int* status_out);

/* Self-test of the bounded device-side waits: one warp waits on a shared-memory barrier that nothing ever
 * completes, with the wait every kernel of this library uses.  Returns KVC_ERR_TIMEOUT when the wait gave up
 * as designed (after about a second) and KVC_OK if it returned as complete (a defect); the CUDA context stays
 * usable either way.  Allocates and frees 4 bytes of device memory and synchronises `stream`. */
KVC_API int kvc_selftest_bounded_wait(void* stream);

/* Collapse of a factored key reconstructor, once per (layer, ratio) before kvc_layer_create.  Sec. 3.1 describes the
 * reconstructor f_theta as a two-layer network while Alg. 1 (step 2) applies a single matrix theta[h] of m x n per KV
 * head to the compressed scores; the two agree when both layers are linear along the token axis, and then
 *   theta[h] = W1[h] W2[h],   W1: DEVICE [H_kv][m][k],  W2: DEVICE [H_kv][k][n],  theta_out: DEVICE [H_kv][m][n],
 * all contiguous, of type `dtype`, caller-owned; theta_out must not overlap the inputs.  fp32 accumulation, one rounding
 * to `dtype`.  m = kvc_retained_len(n, ratio); k >= 1 is the hidden width.  Asynchronous on `stream`; no allocation.
 * Errors: KVC_ERR_ARG (null pointer), KVC_ERR_SHAPE (a size < 1 or a grid dimension beyond 65535), KVC_ERR_DTYPE,
 * KVC_ERR_CUDA (launch failure). */
KVC_API int kvc_collapse_theta(const void* W1, const void* W2, int H_kv, int m, int k, int n, kvc_dtype dtype,
                               void* theta_out, void* stream);

/* Integer maps as the device path uses them: idx_out: HOST [H_kv][m] retained indices per KV head, read back
 * from the device copy the kernels index with; group_out: HOST [R*n][2] = (block r, offset i) of vision token
 * t = r*n + i (the Reshape of Alg. 1 step 1), written on the device by a kernel that uses the row arithmetic of
 * the key selection and copied back.  Either may be NULL.  Synchronous; allocates and frees a temporary of
 * 8*R*n bytes when group_out is given. */
KVC_API int kvc_export_maps(const kvc_layer* layer, int R, int32_t* idx_out, int32_t* group_out);

/* Retained length m and the row stride (in elements) of internal score buffers. */
KVC_API int kvc_layer_m(const kvc_layer* layer);

KVC_API const char* kvc_strerror(int status);

/* Text of the CUDA runtime error behind the calling thread's most recent KVC_ERR_CUDA ("no error" if none). */
KVC_API const char* kvc_last_cuda_error(void);

/* ---- optional instrumentation (measurement only; the paper has no counterpart) -------------
 * While profiling is on, every kernel the library launches is bracketed by two CUDA events
 * recorded on the launching stream, until max_launches brackets have been used.  Global,
 * not thread-safe, and meant for benchmarks: the events serialise nothing but add a little
 * launch work.  kvc_profile_read sums, for one kernel id, the elapsed time of its brackets;
 * call it after the stream has been synchronised.  kvc_profile_start allocates host-side
 * event objects only. */
typedef enum {
  KVC_KERNEL_SCORES = 0,          /* Alg. 1 step 1 + text logits  */
  KVC_KERNEL_EXPAND = 1,          /* Alg. 1 steps 2-3             */
  KVC_KERNEL_OUTPUT = 2,          /* Alg. 1 step 4 + text values  */
  KVC_KERNEL_GATHER_KEYS = 3,     /* key row selection            */
  KVC_KERNEL_PROJECT_VALUES = 4,  /* value centre + project       */
  KVC_KERNEL_MERGE = 5,           /* log-sum-exp merge of partials */
  KVC_KERNEL_COMBINE = 6,         /* n-split partials of Alg. 1 step 3 combined per row */
  KVC_KERNEL_FUSED = 7,           /* Alg. 1 steps 1-4 + text + normalisation in one kernel (bf16) */
  KVC_KERNEL_FUSED_TC = 8,        /* the same kernel with steps 2-3 on tcgen05 / tensor memory (see kvc_layer_create) */
  KVC_KERNEL_FUSED_PAIR = 9,      /* the tensor-memory kernel run by clusters of two CTAs per (sequence, KV head) */
  KVC_KERNEL_SPLIT_SCORES = 10,   /* three-kernel bf16 path: Alg. 1 step 1, one pass over K_tilde */
  KVC_KERNEL_SPLIT_EXPAND = 11,   /* its steps 2-3 on tcgen05, per 128 expansion rows and range of the n axis; the text rows on idle SMs */
  KVC_KERNEL_SPLIT_OUTPUT = 12,   /* its step 4 and the normalisation, one pass over V_tilde, merged with the text partials */
  KVC_KERNEL_RESIDENT = 13,       /* one-kernel bf16 path for short blocks whose theta and U stay in shared memory */
  KVC_KERNEL_COUNT = 14
} kvc_kernel_id;
KVC_API int kvc_profile_start(int max_launches);
KVC_API int kvc_profile_stop(void);
KVC_API int kvc_profile_read(int kernel_id, double* total_ms, long long* launches);
KVC_API const char* kvc_kernel_name(int kernel_id);

#ifdef __cplusplus
}
#endif
#endif /* KVC_H_ */
