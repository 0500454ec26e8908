/*
 * ckv.h -- C ABI of libckv: the end-of-prefill KV retention pass of CompilerKV
 * (arxiv 2602.08686) as hand-written sm_100a CUDA kernels for one B200.
 *
 * Notation: L = prompt length (the paper's T), W = observation-window size
 * |Omega| (the last W prompt positions), n = L - W = prefix length, H = query
 * heads, Hkv = KV heads, G = H / Hkv (query head h reads KV head h / G),
 * d = head_dim, B = rows kept per KV head on average (window included).
 * A "unit" is one (sequence, layer) pair; a call processes Nu independent units.
 *
 * General rules for every entry point
 *   - Every data pointer is a DEVICE pointer unless the argument name ends in
 *     `_host`.  `shape` and `params` are HOST structs read before the call returns.
 *   - The caller owns every buffer.  The library allocates no device memory and
 *     keeps no per-call state; work space is passed in (`ws`, `ws_bytes`, at
 *     least ckv_workspace_bytes(), 256-byte aligned).  What the library does keep,
 *     per process: the defaults of the scheduling settings (ckv_set_score_path,
 *     ckv_set_tunable; results do not depend on them, and a call can carry its own in
 *     params->tuning), a launch counter, and per-device constants it looks up once
 *     (driver entry point, resident CTAs, the address of the fixed scratch); per calling
 *     thread: the default event pair of ckv_set_scan_events.
 *   - Calls are asynchronous on `stream` (a cudaStream_t passed as void*; NULL is
 *     the default stream) and return after the last launch was queued.
 *   - Errors are return codes.  Argument errors are found on the host before
 *     anything is launched (CKV_ERR_INVALID_ARG / UNSUPPORTED / WORKSPACE); a CUDA
 *     launch error gives CKV_ERR_CUDA.  A device-side wait that ran out of its
 *     time limit (2 s unless changed with ckv_set_tunable) is recorded in the work
 *     space's status word, stays there over later calls, and is read back -- and
 *     cleared -- by ckv_device_status().
 *   - Preconditions that are not checked: inputs are finite, head_w >= 0.
 *   - Layouts: q_win [Nu, H, W, d], k and v [Nu, Hkv, L, d]; the last dimension is
 *     contiguous and the other strides are given in ELEMENTS in ckv_shape; every row
 *     must start on a 16-byte boundary; a stride of zero over an extent above one (a
 *     broadcast view) is refused.  All outputs are dense.
 */
#ifndef CKV_H_
#define CKV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  CKV_OK = 0,
  CKV_ERR_INVALID_ARG = 1, /* null / misaligned pointer, inconsistent shape or parameter */
  CKV_ERR_UNSUPPORTED = 2, /* valid but not implemented: head_dim != 128, window > 64, Hkv > 64, ... */
  CKV_ERR_WORKSPACE = 3,   /* ws is null, misaligned or shorter than ckv_workspace_bytes() */
  CKV_ERR_CUDA = 4,        /* a CUDA runtime call or launch failed */
  CKV_ERR_TIMEOUT = 5      /* a bounded device-side wait expired (see ckv_device_status) */
} ckv_status;

typedef enum { CKV_BF16 = 0, CKV_F32 = 1 } ckv_dtype;
typedef enum { CKV_POOL_NONE = 0, CKV_POOL_MAX = 1, CKV_POOL_AVG = 2 } ckv_pool;

typedef struct {
  int32_t n_units;    /* Nu >= 1 */
  int32_t n_q_heads;  /* H, a multiple of n_kv_heads */
  int32_t n_kv_heads; /* Hkv <= 64 */
  int32_t head_dim;   /* d; must be 128 */
  int32_t seq_len;    /* L >= window */
  int32_t window;     /* W in [1, 64] */
  int32_t dtype;      /* ckv_dtype of q_win, k, v and of k_out, v_out */
  int32_t reserved_;  /* set to 0 */
  int64_t q_stride_unit, q_stride_head, q_stride_row;  /* elements */
  int64_t kv_stride_unit, kv_stride_head, kv_stride_tok; /* elements; shared by k and v */
} ckv_shape;

/* Optional per-call settings of how the work is scheduled (never of what is computed: the results do not depend
 * on them).  A field of -1 (a null event) takes the process-wide default that ckv_set_score_path / ckv_set_tunable
 * (for the events: the calling thread's ckv_set_scan_events pair) last set.  Calls on different threads or streams
 * may carry different settings. */
typedef struct {
  int32_t score_path;   /* -1, or as ckv_set_score_path: 0 automatic, 1 plain kernels, 2 tensor-core kernel required */
  int32_t run_tiles;    /* -1, or 1..64 */
  int32_t l2_hints;     /* -1, 0, 1 */
  int32_t group_fuse;   /* -1, 0, 1 */
  int32_t pdl;          /* -1, 0, 1 */
  int32_t reserved_;    /* set to 0 */
  void* scan_start_event;   /* cudaEvent_t pair recorded around the tensor-core scan of this call, or NULL */
  void* scan_stop_event;
} ckv_tuning;

typedef struct {
  int32_t pool_kind;        /* ckv_pool */
  int32_t pool_size;        /* odd, 1..15; 1 (or CKV_POOL_NONE) is the paper's un-pooled score */
  int32_t budget_per_head;  /* B >= 1: rows kept per KV head on average, window included; the unit's
                               heads share Hkv * min(B, L) rows.  B >= L keeps everything (FullKV). */
  int32_t floor_per_head;   /* f >= 0: least number of PREFIX rows any KV head keeps; f <= B - W */
  int32_t n_buckets;        /* size of one row of the threshold table */
  int32_t bucket_override;  /* -1: bucket from the entropy of the unit's window mass; else that bucket */
  int64_t head_w_stride_unit; /* elements between the head_w rows of consecutive units; 0 = one row for all */
  int64_t sens_stride_unit;   /* same for the threshold table */
  int32_t value_norm;       /* 1: ckv_compress multiplies the scores by the value-norm ratio rho of Eq. 4
                               (see ckv_vnorm); 0: u = alpha, the paper's ablation without it */
  float value_norm_eps;     /* the eps of Alg. 1 (B), >= 0 */
  int32_t shared_elastic;   /* 0: one index set per KV head, budgets clamped to sum to Hkv * B (the default);
                               1: the paper's own selection -- Eq. 6's maximum over ALL heads of the unit, Eq. 8's
                               elastic pool (every candidate if at most B - W of them, else the Top-(B - W)), one
                               set shared by the unit's KV heads.  budgets[g] = W + kept are then equal for all g
                               and may be smaller than B; rows of k_out, v_out, indices past offsets[u,Hkv] are
                               left untouched.  ckv_compress applies it; staged callers run ckv_unit_max on the
                               scores before ckv_budget. */
  int32_t global_alpha;     /* 1: the paper's prompt-wide window mass (Alg. 1 (A)): the attention is averaged over all
                               layers and heads of the prompt before the window sum, so alpha, and the entropy that picks
                               the threshold, are one per prompt; see ckv_prompt_mass / ckv_global_scores.  0 (default):
                               per query head of the unit */
  int32_t units_per_prompt; /* with global_alpha: units [s N, (s+1) N) of the call belong to prompt s (its layers);
                               N >= 1 divides n_units.  Ignored otherwise (0 allowed) */
  int32_t reserved_;        /* set to 0 */
  /* The threshold table as the paper indexes it (Sec. 4.3; Alg. 1 (D)): tau = T_gate[l, b_ent, b_ppl, B_l].
     A non-null gate_coords switches it on.  `sens` is then the dense table
     [n_gate_layers][n_buckets][n_ppl_bins][n_budget_levels] fp32 shared by all units (sens_stride_unit must be 0),
     n_buckets counts the entropy bins (20 in the paper, with 4 perplexity bins), b_ent is the unit's entropy bin as
     above, and gate_coords [Nu,3] int32 (DEVICE pointer; a HOST pointer for ckv_compress_host) gives per unit the
     layer row l, the perplexity bin b_ppl of its prompt -- the caller's: Eq. 7's perplexity needs the language
     model's logits -- and the index of its budget level.  Coordinates outside the table are clamped into it. */
  int32_t n_gate_layers;    /* >= 1 with gate_coords; table rows along the layer axis (ckv_gate_depth_map_host maps a
                               table compiled for another depth) */
  int32_t n_ppl_bins;       /* >= 1 with gate_coords */
  int32_t n_budget_levels;  /* >= 1 with gate_coords */
  int32_t reserved2_;       /* set to 0 */
  const int32_t* gate_coords;
  const ckv_tuning* tuning; /* HOST pointer read before the call returns, or NULL for the defaults */
} ckv_params;

/* Bytes of work space any entry point needs for this problem (0 on invalid arguments). */
size_t ckv_workspace_bytes(const ckv_shape* shape, const ckv_params* params);
/* Bytes that ckv_score alone needs: the leading sections of that work space (0 on invalid arguments).  This is
 * also what a problem must fit into for ckv_score_noalloc. */
size_t ckv_score_workspace_bytes(const ckv_shape* shape, const ckv_params* params);

/*
 * Window-score scan and head-table weighting (Sec. 3 softmax; Eq. 4's window mass alpha; Eq. 6's
 * weighted max over heads, taken inside each GQA group; 1-D pooling is an argument the paper does
 * not have).  For every unit and query head h:
 *   s[i,t]  = q_win[h,i] . k[h/G,t] / sqrt(d)   for window row i (position n+i) and keys t <= n+i
 *   A[i,:]  = softmax(s[i,:]);   c_h[t] = sum_i A[i,t];   alpha_h[t] = (L/W) c_h[t]
 *   P_h     = pool(alpha_h[0:n])  (centred, stride 1; MAX ignores positions outside [0,n), AVG
 *             counts them as zeros and divides by pool_size)
 * Outputs: scores [Nu,Hkv,n] fp32, scores[g,t] = max_{h in group g} head_w[h] * P_h[t];
 *          colmass [Nu,L] fp32, colmass[t] = sum_h c_h[t] over all H heads (window columns included).
 * head_w: [H] fp32 per unit (params->head_w_stride_unit apart).
 */
ckv_status ckv_score(const ckv_shape* shape, const ckv_params* params, const void* q_win, const void* k,
                     const float* head_w, float* scores, float* colmass, void* ws, size_t ws_bytes,
                     void* stream);

/*
 * Risk coordinate, threshold lookup and per-head budgets (Eq. 7's attention entropy; the gate
 * lookup of Sec. 4.3 / Alg. 1 (D); Eq. 8's candidate set; the clamp to the total budget).
 *   p[t] = colmass[t] / (W H);  entropy = -sum_t p ln p;  bucket = min(n_buckets-1,
 *   floor(n_buckets * entropy / ln L)) unless overridden;  tau = sens[bucket];
 *   count_g = #{t < n : scores[g,t] >= tau};  demand_g = clamp(count_g, max(f,1), n);
 *   the Hkv (B - W) prefix rows of the unit are split in proportion to the demands with every
 *   share clamped to [f, n] (water-filling in exact integer arithmetic; shares rounded down, the
 *   remainder handed out by largest fractional part, ties to the lowest head);
 *   budgets[g] = W + share_g, so sum_g budgets[g] = Hkv B.  B >= L gives budgets[g] = L.
 * Outputs: budgets [Nu,Hkv] int32; offsets [Nu,Hkv+1] int32 (exclusive prefix sums of budgets);
 *          bucket [Nu] int32; entropy [Nu] fp32.  sens: [n_buckets] fp32 per unit.
 */
ckv_status ckv_budget(const ckv_shape* shape, const ckv_params* params, const float* scores,
                      const float* colmass, const float* sens, int32_t* budgets, int32_t* offsets,
                      int32_t* bucket, float* entropy, void* ws, size_t ws_bytes, void* stream);

/*
 * Value-norm ratio of the stabilised utility (Eq. 4, Alg. 1 (B)), per unit and KV head (under GQA the
 * values belong to the KV head, so a group's query heads share it):
 *   r[t] = |v[t,:]|_2 over all L tokens;  rho[t] = r[t] / (mean_t r[t] + value_norm_eps)
 * rho [Nu,Hkv,L] fp32 (output).  When scores_or_null [Nu,Hkv,n] is given, scores[g,t] *= rho[g,t] in
 * place for the prefix: Eq. 4's u = alpha * rho applied after the pooling and, because rho >= 0 is
 * common to the group, equal to applying it before Eq. 6's maximum.  v is read once (Hkv L d elements
 * per unit).  Runs whatever params->value_norm says; that flag only steers ckv_compress.
 */
ckv_status ckv_vnorm(const ckv_shape* shape, const ckv_params* params, const void* v, float* rho,
                     float* scores_or_null, void* ws, size_t ws_bytes, void* stream);

/*
 * Decode-side check of the compressed cache (the setting of Prop. 4.1; not part of the retention pass): softmax
 * attention of n_dec decode queries per query head -- queries that come after the prompt and see every row -- over
 *   compressed == 0: all L rows of k, v [Nu,Hkv,L,d] (strides of `shape`);
 *   compressed == 1: the rows the pass kept; k, v are then k_out, v_out [Nu, Hkv min(B,L), d] and head g of unit u
 *                    owns budgets[u,g] rows from row offsets[u,g].
 * q_dec [Nu,H,n_dec,d] dense, in the dtype of `shape`; (H / Hkv) * n_dec <= 32, else CKV_ERR_UNSUPPORTED.
 * out [Nu,H,n_dec,d] fp32 = softmax(q k^T / sqrt d) v;  lse [Nu,H,n_dec] fp32 = ln sum_t exp(q . k_t / sqrt d).
 * With both runs, the discarded mass of the proposition is m = 1 - exp(lse_compressed - lse_full), the compressed
 * output is the attention under the renormalised restriction p~, and |p - p~|_1 = 2 m.
 */
ckv_status ckv_attend(const ckv_shape* shape, const ckv_params* params, const void* q_dec, int32_t n_dec,
                      const void* k, const void* v, int32_t compressed, const int32_t* budgets, const int32_t* offsets,
                      float* out, float* lse, void* ws, size_t ws_bytes, void* stream);

/*
 * Diagnostic of Prop. 4.1 on the observation-window rows (they stand in for decode queries): the attention mass
 * that survives the selection,
 *   kept[u,h,i] = sum over the retained positions t of KV head h/G that row i can see of A^h[n+i, t],
 * so that m = 1 - kept is the discarded mass, |p - p~|_1 = 2 m for the renormalised restriction p~, and
 * eps_tail = sqrt(mean_i m^2) enters the Frobenius bound of the proposition.  Computed from the gathered keys k_out
 * (so it also checks what ckv_gather wrote) and the softmax normalisers that the last ckv_score / ckv_compress
 * call on this work space left in it; indices, budgets, offsets, k_out as produced by that pass.
 * kept [Nu,H,W] fp32.  Not part of the retention pass itself.
 */
ckv_status ckv_kept_mass(const ckv_shape* shape, const ckv_params* params, const void* q_win, const void* k_out,
                         const int32_t* indices, const int32_t* budgets, const int32_t* offsets, float* kept, void* ws,
                         size_t ws_bytes, void* stream);

/*
 * Prompt-global window mass (Alg. 1 (A): A-bar = mean over layers and heads; alpha = (T/W) sum_{j in Omega} A-bar[j,:]),
 * for params->global_alpha.  After ckv_score:
 *   ckv_prompt_mass    pmass[s,t] = sum over the prompt's units in this call of colmass[u,t]; pmass [Nu/N, L] fp32.
 *   ckv_global_scores  alpha_s = (L/W) pmass[s] / (units_total * H);
 *                      scores[u,g,t] = (max_{h in g} head_w[u,h]) * pool(alpha_s)[t]  (alpha >= 0, so Eq. 6's maximum
 *                      over the group is its largest weight), overwriting ckv_score's per-head scores;
 *                      colmass[u,:] = pmass[s,:] / units_total, so that ckv_budget takes one entropy per prompt.
 * units_total is the prompt's number of units on ALL devices (>= units_per_prompt): where a prompt's layers are
 * spread over several GPUs, the caller adds the ranks' pmass arrays between the two calls (the method's one
 * exchange step; paper_2602_08686_b200/sharding.py has the all-reduce).  ckv_compress runs both calls itself with
 * units_total = units_per_prompt.  The value-norm ratio and the selection follow as usual.
 */
ckv_status ckv_prompt_mass(const ckv_shape* shape, const ckv_params* params, const float* colmass, float* pmass,
                           void* stream);
ckv_status ckv_global_scores(const ckv_shape* shape, const ckv_params* params, const float* head_w,
                             const float* pmass, int32_t units_total, float* scores, float* colmass, void* stream);

/*
 * Eq. 6 over all heads of a unit (used by the shared elastic selection): scores[u,g,t] is replaced, for
 * every KV head g, by max_g' scores[u,g',t].  In place.
 */
ckv_status ckv_unit_max(const ckv_shape* shape, const ckv_params* params, float* scores, void* stream);

/*
 * Per-head Top-k (Eq. 8's Top-B branch).  For every unit and KV head g the budgets[g] - W
 * largest of scores[g,0:n] are kept, equal scores resolved toward the lowest index; the kept
 * positions are written in ascending order and followed by the window n .. L-1, which is always
 * retained.  indices [Nu, Hkv * min(B,L)] int32, head g of unit u at row offsets[u,g] of the unit's
 * Hkv * min(B,L) rows.  Of the work space only the status word is used: prefixes longer than 32768
 * are searched by clusters of CTAs, whose bounded exchange wait reports there (ckv_device_status).
 */
ckv_status ckv_select(const ckv_shape* shape, const ckv_params* params, const float* scores,
                      const int32_t* budgets, const int32_t* offsets, int32_t* indices, void* ws,
                      size_t ws_bytes, void* stream);

/*
 * Gather of the retained rows (K~ = K[S], V~ = V[S] of Sec. 3 / Alg. 1 (D)): bit copies.
 * k_out, v_out [Nu, Hkv * min(B,L), d] in the input dtype, rows in the order of `indices`.
 */
ckv_status ckv_gather(const ckv_shape* shape, const ckv_params* params, const void* k, const void* v,
                      const int32_t* indices, const int32_t* offsets, void* k_out, void* v_out,
                      void* stream);

/*
 * The whole pass in one call: score -> budget -> select -> gather on one stream (Alg. 1 (A)-(D)
 * for the per-unit reading described above).  scores_or_null [Nu,Hkv,n] receives the scores when
 * given; bucket_or_null [Nu] and entropy_or_null [Nu] likewise.
 */
ckv_status ckv_compress(const ckv_shape* shape, const ckv_params* params, const void* q_win, const void* k,
                        const void* v, const float* head_w, const float* sens, void* k_out, void* v_out,
                        int32_t* indices, int32_t* budgets, int32_t* offsets, float* scores_or_null,
                        int32_t* bucket_or_null, float* entropy_or_null, void* ws, size_t ws_bytes,
                        void* stream);

/*
 * The whole pass on HOST buffers (pinned memory recommended): copies q_win, k, v, head_w and sens
 * into `staging` (device memory, at least ckv_staging_bytes(), 256-byte aligned), runs
 * ckv_compress, copies k_out, v_out, indices, budgets and offsets back, and synchronises the
 * stream before returning.  Host tensors are dense ([Nu,H,W,d], [Nu,Hkv,L,d], head_w [Nu,H] or [H]
 * by head_w_stride_unit, sens likewise); the strides in `shape` are ignored.
 * V is only gathered (Alg. 1 (D)) unless params->value_norm streams it: when v_host is page-locked memory that the
 * device has mapped (ckv_reads_in_place(v_host) == 1; true of cudaHostAlloc / cudaHostRegister memory on systems
 * with unified addressing), V is not copied at all and the gather reads the kept rows from the host buffer in
 * place, so that of V only Hkv * min(B, L) rows per unit cross the bus.  Pageable memory is copied as a whole.
 */
size_t ckv_staging_bytes(const ckv_shape* shape, const ckv_params* params);
/* 1 if a kernel can read this host buffer in place (see ckv_compress_host), 0 if it would be copied. */
int ckv_reads_in_place(const void* host_pointer);
ckv_status ckv_compress_host(const ckv_shape* shape, const ckv_params* params, const void* q_win_host,
                             const void* k_host, const void* v_host, const float* head_w_host,
                             const float* sens_host, void* k_out_host, void* v_out_host,
                             int32_t* indices_host, int32_t* budgets_host, int32_t* offsets_host,
                             void* staging, size_t staging_bytes, void* ws, size_t ws_bytes, void* stream);

/*
 * ckv_score without a work-space argument, for callers that cannot allocate device memory: code
 * that runs inside another framework's memory plan or under a fixed memory budget, where every
 * byte of HBM was handed out before this library is called and cudaMalloc (or a framework
 * allocator that may fall back to it) is off limits, or too slow, at that point.  The paper has
 * no counterpart to this entry point; it computes exactly what ckv_score computes, with the same
 * kernels, and differs only in where the intermediate data lives.
 *
 * The scratch is a fixed array of CKV_NOALLOC_SCRATCH_BYTES bytes in the library's own device
 * image: every GPU on which the library is loaded holds it from load until the process exits.
 * Only the sections of the work space that the score stage uses count against that size (a little over half
 * of ckv_workspace_bytes(); about 7.5 MB per unit of 32 query heads at L = 32768); larger problems are refused
 * with CKV_ERR_WORKSPACE before anything is launched (use ckv_score with a caller-owned work space for those).
 *   - Nothing is allocated or freed, by the CUDA runtime or otherwise.  The first call on a device
 *     looks up the array's device address (one runtime query, remembered per device); make that
 *     first call outside any stream capture.
 *   - All calls on one device share the array and it keeps whatever the last call left in it; the
 *     entry point clears the few words that must start at zero.  Two calls whose kernels can run at
 *     the same time on one device (different streams without an ordering between them) race on it:
 *     serialise them.
 *   - The device status word lives inside the array: ckv_device_status(NULL, stream) reads it on the
 *     current device.
 * Arguments, layouts, outputs and the remaining error codes are those of ckv_score.
 */
#define CKV_NOALLOC_SCRATCH_BYTES (16u << 20)
ckv_status ckv_score_noalloc(const ckv_shape* shape, const ckv_params* params, const void* q_win,
                             const void* k, const float* head_w, float* scores, float* colmass,
                             void* stream);

/* Synchronises `stream` and returns what device code recorded in the status word of `ws` since the last
 * such call (CKV_OK or CKV_ERR_TIMEOUT), or CKV_ERR_CUDA if the stream is in error.  A recorded code survives
 * later calls on the work space until this function reports it, which also clears it.  ws == NULL reads the
 * fixed scratch of ckv_score_noalloc on the current device.  Work space that no call has used yet reads CKV_OK. */
ckv_status ckv_device_status(const void* ws, void* stream);

/* Diagnostic switch for the window-score scan: 0 = automatic (tensor-core kernel for bf16 inputs with
 * window 16, 32 or 64 and L >= 128, plain kernels otherwise), 1 = always the plain kernels, 2 = require
 * the tensor-core kernel (ckv_score returns CKV_ERR_UNSUPPORTED where it does not apply).  Process-wide default
 * (a call may carry its own in params->tuning);
 * returns the previous setting, or -1 for an invalid value. */
int ckv_set_score_path(int path);

/* Timing hook: when both are non-null cudaEvent_t handles (created with timing enabled, owned by the
 * caller), every later ckv_score / ckv_compress call that runs the tensor-core scan records
 * start_event just before and stop_event just after that kernel's launch, on the call's stream, so
 * that the scan can be timed inside a fused call.  Pass nulls to switch it off.  The pair belongs to the calling
 * thread: calls made from other threads are not affected and record nothing. */
void ckv_set_scan_events(void* start_event, void* stop_event);

/* Diagnostic knobs of the tensor-core scan (process-wide defaults, see ckv_tuning; the scores do not depend on them):
 *   "run_tiles"      key tiles per run, the unit CTAs take work in (1..64, default 16);
 *   "l2_hints"       1 (default): first-pass K loads ask L2 to keep their lines and second-pass loads
 *                    release them; 0: no hints;
 *   "group_fuse"     1 (default): where a KV group's query heads fill one 128-row block and the pooling
 *                    is max or none, the scan itself takes the weighted maximum over the group's heads
 *                    (Eq. 6) and adds their column mass, and the pooling runs on that one row per group;
 *                    the scores are bit-identical to the per-head order of operations for head_w >= 0,
 *                    the column mass may differ in the last bit (heads are added group by group);
 *                    0: always write per-head column sums;
 *   "pdl"            1 (default): the counting, selection and gather kernels are launched with programmatic
 *                    stream serialisation, so each is scheduled while its predecessor drains and waits on the
 *                    device for it to complete; 0: ordinary launches;
 *   "wait_limit_us"  time limit of every bounded device-side wait in microseconds (default 2000000).  A wait
 *                    that runs out makes its kernel wind down and records CKV_ERR_TIMEOUT in the status word;
 *                    the outputs of that call are then incomplete.
 * Returns the previous value, or -1 for an unknown name or a value out of range. */
int ckv_set_tunable(const char* name, int value);

/* Number of kernel launches this process has queued through the library so far. */
int64_t ckv_kernel_launches(void);

/* Host-only: the integer split of P prefix rows over hkv heads used by ckv_budget (demands >= 1,
 * shares in [f, n], f*hkv <= P <= n*hkv), exposed so that it can be checked without a GPU.
 * Returns 0 on success. */
int ckv_allocate_rows_host(int hkv, int64_t n, int64_t f, int64_t P, const int64_t* demands, int64_t* out);

/* Host-only: a table compiled for n_src layers ([n_src][row_elems] fp32, e.g. the gate table with row_elems =
 * n_buckets * n_ppl_bins * n_budget_levels, or the head table with row_elems = H) mapped to a model of n_dst
 * layers by relative depth (the paper's appendix on cross-architecture use: a monotone depth mapping by
 * relative-depth interpolation): target layer l takes the linear interpolation of the source rows around
 * position l (n_src - 1) / (n_dst - 1); first and last layers map onto first and last, equal depths give a copy.
 * dst [n_dst][row_elems].  Returns 0 on success, 1 on invalid arguments. */
int ckv_gate_depth_map_host(const float* src, int n_src, int n_dst, int64_t row_elems, float* dst);

const char* ckv_status_string(ckv_status status);
int ckv_version(void);

#ifdef __cplusplus
}
#endif
#endif /* CKV_H_ */
