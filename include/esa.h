/*
 * esa.h -- C ABI of the B200 (sm_100a) library for one step of Efficient
 * Selective Attention (ESA, arXiv 2502.14477).
 *
 * One step (Section 3.1 of the paper), for the current chunk C that follows t
 * cached tokens:
 *   esa_compress_keys  Eq. 5   k' = f_k(k): compressed keys of C appended to the cache
 *   esa_select         Eq. 5   q' = f_q(q) for the queries of C
 *                      Eq. 6   S[c,m] = q'_c . k'_m over the middle tokens M
 *                      Eq. 4   s_m = max_c ( S[c,m] - max_m' S[c,m'] )
 *                      Eq. 8   s'_j = max of s over [j-eps, j+eps] clipped to M
 *                      Eq. 2   the k largest s' (ties: lowest index), ascending positions
 *   esa_attend         Eq. 1 / Algorithm 1: softmax attention of the queries of C over
 *                      I u M_k u L u C (C causal), all heads sharing one selection
 *
 * Token partition (Section 3.1): with l_I = l_init and l_L = l_local,
 *   I = [0, i_end), M = [i_end, m_end), L = [m_end, t), C = [t, t + l_C)
 *   i_end = min(l_I, t), m_end = max(i_end, t - l_L), k_eff = min(top_k, m_end - i_end).
 *
 * Conventions
 *   - Every function returns an esa_status.  Argument, shape and capacity errors are
 *     found on the host before anything is launched and leave all outputs untouched.
 *   - "device" pointers are CUDA device memory owned by the caller; "host" pointers are
 *     ordinary host memory read before the call returns.  The library never frees or
 *     reallocates caller memory.  Tensors are dense, row-major, bf16 unless noted.
 *   - *_async variants only enqueue work on the given CUDA stream (a cudaStream_t passed
 *     as void*) and return without synchronising.  The plain variants run on the legacy
 *     default stream and return after the work has finished.
 *   - A context owns device workspace shared by its calls: esa_select and esa_attend calls
 *     on the same context must be ordered (one stream, or externally synchronised); use one
 *     context per stream for them.  esa_compress_keys and esa_append_kv touch none of that
 *     workspace (they read the weights and write caller memory): they may run on another
 *     stream beside a select or attend of the same context, as long as the caller orders
 *     them against the calls that read the rows they write (the selection reads rows of M
 *     only, the attention reads every row up to the end of the current chunk).
 *   - Device-side problems (a bounded wait that ran out, a selected position outside the
 *     middle tokens) are recorded in a status word read by esa_last_device_status; kernels
 *     never trap and never read outside the caches.
 *   - The compressed-key cache is caller memory with library-defined contents: row p of
 *     sequence b is k'_p (bf16, d_c values).  n_prev[b] is the only record of its length.
 */
#ifndef ESA_H_
#define ESA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct esa_ctx esa_ctx;

typedef enum {
    ESA_OK = 0,
    ESA_ERR_INVALID_ARG = 1,  /* null pointer, negative size, bad handle            */
    ESA_ERR_SHAPE = 2,        /* a dimension the kernels do not support               */
    ESA_ERR_CAPACITY = 3,     /* exceeds max_chunk / max_batch / max_tokens           */
    ESA_ERR_CUDA = 4,         /* a CUDA runtime call failed                           */
    ESA_ERR_TIMEOUT = 5,      /* a bounded device-side wait ran out                   */
    ESA_ERR_UNSUPPORTED = 6,  /* valid request the library does not implement         */
    ESA_ERR_STATE = 7,        /* call order: compressors not set                      */
    ESA_ERR_INDEX = 8         /* a selected position passed to esa_attend lay outside M */
} esa_status;

/* Hyper-parameters of the step (paper symbols in comments) and capacities. */
typedef struct {
    int32_t n_q_heads;     /* H                                                        */
    int32_t n_kv_heads;    /* H_G, divides H                                           */
    int32_t head_dim;      /* d: 64 or 128                                             */
    int32_t d_c;           /* d' : 32, 64 or 128                                       */
    int32_t l_init;        /* l_I                                                      */
    int32_t l_local;       /* l_L                                                      */
    int32_t top_k;         /* k                                                        */
    int32_t eps;           /* proximity distance of Eq. 8, 0..15                       */
    int32_t max_chunk;     /* largest l_C of any call                                  */
    int32_t max_batch;     /* largest B of any call, <= 64                             */
    int64_t max_tokens;    /* rows per sequence in every cache, < 2^31                 */
    float softmax_scale;   /* 0 selects 1/sqrt(head_dim)                               */
} esa_config;

/* Human-readable name of a status code (static storage). */
const char* esa_status_string(esa_status s);

/* Bytes of device workspace esa_create will allocate for this configuration
 * (0 if the configuration is invalid). */
size_t esa_workspace_bytes(const esa_config* cfg);

/* Create a context on the current CUDA device; allocates its workspace there. */
esa_status esa_create(const esa_config* cfg, esa_ctx** out);
esa_status esa_destroy(esa_ctx* ctx);

/* Eq. 5: install the two linear compressors.  Host fp32 pointers:
 * Wq [d_c, H*d], Wk [d_c, H_G*d] (row-major; a key compressor defined on H repeated
 * heads folds to this shape by summing each group's columns), bq/bk [d_c] or NULL for
 * no bias.  Weights are rounded once to bf16 (round-to-nearest-even) and copied to
 * the device; biases stay fp32.  Synchronous copies on the default stream: work of this
 * context that is still in flight on a non-blocking stream must be waited for first. */
esa_status esa_set_compressors(esa_ctx* ctx, const float* Wq, const float* bq,
                               const float* Wk, const float* bk);

/* Appends the rows of the current chunk to the caller's K and V caches
 * (Section 3.1: keys and values of every token are cached; nothing is evicted).
 * K_new, V_new: device [B, n_new, H_G, d].  K_cache, V_cache: device
 * [B, max_tokens, H_G, d]; rows [n_prev[b], n_prev[b]+n_new) of sequence b are written.
 * n_prev: host [B].  ESA_ERR_CAPACITY if n_prev[b]+n_new > max_tokens. */
esa_status esa_append_kv(esa_ctx* ctx, int32_t B, const void* K_new, const void* V_new,
                         int32_t n_new, void* K_cache, void* V_cache, const int64_t* n_prev);
esa_status esa_append_kv_async(esa_ctx* ctx, int32_t B, const void* K_new, const void* V_new,
                               int32_t n_new, void* K_cache, void* V_cache,
                               const int64_t* n_prev, void* stream);

/* Eq. 5 for keys: kc_cache[b, n_prev[b] + i, :] = bf16( Wk . K_new[b, i, :, :] + bk ),
 * fp32 accumulation.  K_new: device [B, n_new, H_G, d].  kc_cache: device
 * [B, max_tokens, d_c].  n_prev: host [B].  n_new <= max(max_chunk, 4096) per call. */
esa_status esa_compress_keys(esa_ctx* ctx, int32_t B, const void* K_new, int32_t n_new,
                             void* kc_cache, const int64_t* n_prev);
esa_status esa_compress_keys_async(esa_ctx* ctx, int32_t B, const void* K_new, int32_t n_new,
                                   void* kc_cache, const int64_t* n_prev, void* stream);

/* Eq. 5 (queries), Eq. 6, Eq. 4, Eq. 8, Eq. 2.  Q_cur: device [B, l_C, H, d].
 * kc_cache must hold k' for positions [0, n_prev[b]) (only M is read).
 * Outputs: idx_out device int32 [B, top_k]: the first n_sel_out[b] entries of row b are
 * the selected absolute positions, ascending; n_sel_out device int32 [B] = k_eff.
 * When k_eff equals the number of middle tokens all of M is returned without scoring.
 * Scores are fp32; q' is rounded to bf16 like k'. */
esa_status esa_select(esa_ctx* ctx, int32_t B, const void* Q_cur, int32_t l_C,
                      const void* kc_cache, const int64_t* n_prev,
                      int32_t* idx_out, int32_t* n_sel_out);
esa_status esa_select_async(esa_ctx* ctx, int32_t B, const void* Q_cur, int32_t l_C,
                            const void* kc_cache, const int64_t* n_prev,
                            int32_t* idx_out, int32_t* n_sel_out, void* stream);

/* Selection on full-dimension scores, the two variants the paper compares the compressed
 * scores with (no compressors involved; K_cache is read instead of the compressed-key cache):
 *   ESA_SCORE_UNIFORM   Eq. 3: f_s(m; c) = sum over the H heads of q_{h,c} . k_{h,m}, then Eq. 4, 8, 2
 *                       ("uniform" in Section 4.3: the method without dimensionality reduction; its
 *                       selection is the ground truth of the recall measurement of Fig. 3)
 *   ESA_SCORE_PER_HEAD  Section 4.3 "individual": Eq. 4 per head, a token's score is the largest of
 *                       its H head scores; then Eq. 8 and Eq. 2
 * Q_cur: device [B, l_C, H, d]; K_cache: device [B, max_tokens, H_G, d] (rows of M are read).
 * Outputs as for esa_select.  bf16 products, fp32 accumulation over all heads and dimensions. */
typedef enum { ESA_SCORE_UNIFORM = 0, ESA_SCORE_PER_HEAD = 1 } esa_score_mode;
esa_status esa_select_full(esa_ctx* ctx, int32_t B, const void* Q_cur, int32_t l_C, const void* K_cache,
                           const int64_t* n_prev, int32_t mode, int32_t* idx_out, int32_t* n_sel_out);
esa_status esa_select_full_async(esa_ctx* ctx, int32_t B, const void* Q_cur, int32_t l_C, const void* K_cache,
                                 const int64_t* n_prev, int32_t mode, int32_t* idx_out, int32_t* n_sel_out,
                                 void* stream);

/* Eq. 1 / Algorithm 1.  Q_cur: device [B, l_C, H, d].  K_cache, V_cache: device
 * [B, max_tokens, H_G, d] that already hold C at rows [n_prev[b], n_prev[b]+l_C).
 * idx: device int32 [B, top_k] and n_sel: device int32 [B] as written by esa_select
 * (positions must lie in M, ascending order is not required; a position outside M is
 * replaced by the nearest position of M, so that no row outside the caches is read, and
 * ESA_ERR_INDEX is recorded in the device status word).  O: device [B, l_C, H, d]
 * bf16.  Query head h reads key/value head h / (H/H_G).  Query c of the chunk attends
 * every I, selected-M and L key and the keys of C at chunk offsets <= c; bf16 products,
 * fp32 softmax and accumulation.
 *
 * Ordering.  The call is ordered after everything enqueued on its stream before it, with one
 * exception that the caller must know.  A call that is the first esa_attend* on `stream` after an
 * esa_select* made through the same context on the same stream (the usual step: select, then
 * attend) reads the cache rows older than the chunk (positions < n_prev[b]: the rows of I and L)
 * while the selection kernels may still be running, and only then waits for the work ahead of it
 * in the stream; those rows do not depend on the selection (Section 3.2: I and L are always kept).
 * Between such a pair of calls the caller therefore enqueues nothing on the stream that writes K
 * or V rows at positions < n_prev[b]; rows of the chunk itself (esa_append_kv), idx, n_sel and
 * anything else may be written there.  Any other esa_attend call starts all of its reads after
 * the preceding work of the stream.  The two orders add the same terms in another order: results
 * agree to the rounding of bf16 (not bit for bit). */
esa_status esa_attend(esa_ctx* ctx, int32_t B, const void* Q_cur, int32_t l_C,
                      const void* K_cache, const void* V_cache, const int64_t* n_prev,
                      const int32_t* idx, const int32_t* n_sel, void* O);
esa_status esa_attend_async(esa_ctx* ctx, int32_t B, const void* Q_cur, int32_t l_C,
                            const void* K_cache, const void* V_cache, const int64_t* n_prev,
                            const int32_t* idx, const int32_t* n_sel, void* O, void* stream);

/* Section 3.2 (position encoding) / Algorithm 1 with two encodings of the same tokens.  The
 * paper attends I and M_k at one fixed distance (the queries of C encoded at a fixed position
 * w, those keys at position 0) and L and C at their true relative positions, and normalises
 * over both parts together.  The rotation itself stays with the caller; this call takes the two
 * encodings as separate tensors:
 *   Q_cur       device [B, l_C, H, d]             queries used against L and C
 *   Q_far       device [B, l_C, H, d] or NULL     queries used against I and M_k   (NULL: Q_cur)
 *   K_cache     device [B, max_tokens, H_G, d]    keys read for L and C
 *   K_far_cache device [B, max_tokens, H_G, d] or NULL   keys read for I and M_k  (NULL: K_cache)
 * One softmax spans the logits of both parts (Algorithm 1's merge of its two partial results by
 * their normalisers); values come from V_cache for every key.  Everything else is as for
 * esa_attend, which is this call with both optional tensors NULL. */
esa_status esa_attend_two_position(esa_ctx* ctx, int32_t B, const void* Q_cur, const void* Q_far, int32_t l_C,
                                   const void* K_cache, const void* K_far_cache, const void* V_cache,
                                   const int64_t* n_prev, const int32_t* idx, const int32_t* n_sel, void* O);
esa_status esa_attend_two_position_async(esa_ctx* ctx, int32_t B, const void* Q_cur, const void* Q_far, int32_t l_C,
                                         const void* K_cache, const void* K_far_cache, const void* V_cache,
                                         const int64_t* n_prev, const int32_t* idx, const int32_t* n_sel, void* O,
                                         void* stream);

/* Appendix "Model Loading": the K/V cache offloaded to host memory, the compressed keys on
 * the GPU, and only the attended rows brought onto the GPU at every step (the paper's
 * single-GPU mode for contexts of 700k+ tokens).  esa_attend with host-resident caches:
 *   K_host, V_host   [B, max_tokens, H_G, d] in page-locked host memory that the device can
 *                    address (cudaHostAlloc / cudaHostRegister; pass the device-side pointer,
 *                    which equals the host pointer under unified addressing).  They already
 *                    hold C at rows [n_prev[b], n_prev[b] + l_C).
 *   K_stage, V_stage device [B, stage_rows, H_G, d] scratch owned by the caller, stage_rows >=
 *                    l_I + top_k + l_L + l_C: the rows of I, M_k, L and C are copied there in
 *                    list order by one gather kernel (16-byte reads across PCIe), and the
 *                    attention kernels run on the staged rows.
 * Everything else is as for esa_attend; the result is bit-identical to an esa_attend on
 * device-resident copies of the same caches that does not follow a selection (the staged rows
 * are written by the gather kernel just ahead, so this call never reads rows early: see
 * "Ordering" above).  ESA_ERR_CAPACITY if stage_rows is too small. */
esa_status esa_attend_host_kv(esa_ctx* ctx, int32_t B, const void* Q_cur, int32_t l_C, const void* K_host,
                              const void* V_host, const int64_t* n_prev, const int32_t* idx, const int32_t* n_sel,
                              void* K_stage, void* V_stage, int64_t stage_rows, void* O);
esa_status esa_attend_host_kv_async(esa_ctx* ctx, int32_t B, const void* Q_cur, int32_t l_C, const void* K_host,
                                    const void* V_host, const int64_t* n_prev, const int32_t* idx, const int32_t* n_sel,
                                    void* K_stage, void* V_stage, int64_t stage_rows, void* O, void* stream);

/* (No counterpart in the paper: an integration convenience.)
 * esa_attend for small chunks -- l_C * (H / H_G) <= 64 rows, the decode case -- that needs
 * neither a context nor any allocation.  It is for callers that may not allocate device
 * memory once they are running: a serving loop in which the implicit device-wide
 * synchronisation of cudaMalloc / cudaFree would stall every other stream, or a host
 * application that has already handed all device memory to its own pool so that a driver
 * allocation would fail.  esa_create allocates a workspace and therefore does not suit
 * them; this entry point calls no allocating routine at all.
 *
 * The partial results of the key-list splits go to a fixed 8 MiB array inside the library
 * image (held on every GPU that loads the library, until the process exits).  A call is
 * refused with ESA_ERR_CAPACITY when the chunk has more than 64 rows per key/value head,
 * or when B * H_G * rows * (head_dim + 2) * 4 floats exceed the array (four splits is the
 * least it will run with); e.g. B = 8, H_G = 8, l_C = 1, H / H_G = 4, head_dim = 128 uses
 * 0.13 MiB per split.  Used fields of cfg: n_q_heads, n_kv_heads, head_dim, l_init,
 * l_local, top_k, max_tokens, softmax_scale.  All other arguments are as for
 * esa_attend_async; work is only enqueued on `stream`.
 *
 * The first call on each device looks up the array's device address; make that call with
 * the device current and before any stream capture is started on that device.  Host threads
 * may make that first call at the same time (the look-up is serialised inside the library).  Every call
 * on a device shares the one array: calls that may overlap on the GPU (different streams,
 * no ordering between them) race on it and give wrong results; order them.  Nothing in the
 * array has to be cleared between calls -- each call writes every slot it later reads. */
esa_status esa_attend_noalloc(const esa_config* cfg, int32_t B, const void* Q_cur, int32_t l_C,
                              const void* K_cache, const void* V_cache, const int64_t* n_prev,
                              const int32_t* idx, const int32_t* n_sel, void* O, void* stream);

/* Eq. 7: fitting the two compressors.  A trainer holds W_q [d_c, H*d], b_q, W_k [d_c, H_G*d], b_k
 * and their Adam moments on the device (fp32).  One step takes a batch of n query-key pairs
 * (Q_batch device bf16 [n, H, d], K_batch device bf16 [n, H_G, d], n <= batch), forms the full-dimension
 * scores q_c k_m^T of all n x n pairs (Eq. 3), the compressed ones f_q(q_c) . f_k(k_m), the mean
 * squared difference and its gradients, and applies one Adam update (beta 0.9 / 0.999, eps 1e-8,
 * no weight decay; the paper names no optimiser, Section 4.1 gives the learning rate 5e-4, batches
 * of 128 and 10 epochs).  loss_out: device fp32, receives the loss before the update (may be NULL).
 * Used fields of cfg: n_q_heads, n_kv_heads, head_dim, d_c.  esa_fit_set_weights installs host fp32
 * initial values (biases may be NULL = 0) and resets the optimiser; esa_fit_get_weights synchronises
 * the device and copies the current values to host memory (pass them to esa_set_compressors). */
typedef struct esa_fit esa_fit;
esa_status esa_fit_create(const esa_config* cfg, int32_t batch, float lr, esa_fit** out);
esa_status esa_fit_destroy(esa_fit* fit);
esa_status esa_fit_set_weights(esa_fit* fit, const float* Wq, const float* bq, const float* Wk, const float* bk);
esa_status esa_fit_get_weights(esa_fit* fit, float* Wq, float* bq, float* Wk, float* bk);
esa_status esa_fit_step_async(esa_fit* fit, const void* Q_batch, const void* K_batch, int32_t n, float* loss_out,
                              void* stream);
int64_t esa_fit_launch_count(const esa_fit* fit);

/* Diagnostic: copies the pooled scores s' (Eq. 8) of the most recent esa_select of
 * sequence b to host memory dst[0..n) as fp32, n <= number of middle tokens of that
 * call.  Synchronises the given stream.  ESA_ERR_STATE if that call did no scoring. */
esa_status esa_read_pooled_scores(esa_ctx* ctx, int32_t b, float* dst_host, int64_t n,
                                  void* stream);

/* Diagnostic: copies q' (Eq. 5) of the most recent esa_select that scored -- its B * l_C
 * rows of d_c bf16 values, row b * l_C + c for query c of sequence b -- to host memory
 * dst_host[0 .. n_rows * d_c) as raw bf16 bit patterns.  Synchronises the given stream.
 * ESA_ERR_STATE if that call did no scoring, ESA_ERR_CAPACITY if n_rows exceeds its rows. */
esa_status esa_read_compressed_queries(esa_ctx* ctx, void* dst_host, int64_t n_rows, void* stream);

/* Diagnostic of the bounded device-side waits: enqueues a one-thread kernel that waits, for
 * at most limit_cycles SM clock cycles (1 <= limit_cycles <= 2e9, about a second), on a
 * barrier that nothing ever completes.  The wait gives up, ESA_ERR_TIMEOUT is recorded in the
 * status word and the kernel returns: the same path a kernel of the library takes when one of
 * its waits runs out.  Nothing faults and the context stays usable. */
esa_status esa_debug_wait_timeout(esa_ctx* ctx, int64_t limit_cycles, void* stream);

/* Per-kernel timing.  While profiling is on, every kernel the context launches is bracketed by
 * two CUDA events on the launching stream (events are created on first use and reused).  An
 * event between two kernels of a step prevents the second from starting under the first one's
 * tail, so profiled calls run somewhat slower than unprofiled ones: switch it on for sampled
 * calls only.  esa_read_profile waits for the recorded events, adds the elapsed times up per
 * kernel class (esa_kernel_class_count classes, named by esa_kernel_class_name; a class that
 * covers two launches is timed across both) into launches[] / total_ms[] (n_classes entries,
 * at least the class count) and forgets the records. */
int32_t esa_kernel_class_count(void);
const char* esa_kernel_class_name(int32_t cls);
esa_status esa_set_profiling(esa_ctx* ctx, int32_t on);
esa_status esa_read_profile(esa_ctx* ctx, int32_t n_classes, int64_t* launches, double* total_ms);

/* Number of kernels this context has launched since creation (host counter). */
int64_t esa_launch_count(const esa_ctx* ctx);

/* Synchronises the stream, then returns ESA_OK or the error a kernel recorded
 * (and clears the record, together with the merge bookkeeping that an abandoned
 * kernel may have left behind: the context stays usable). */
esa_status esa_last_device_status(esa_ctx* ctx, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* ESA_H_ */
