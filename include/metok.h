/*
 * metok.h -- C ABI of the METok hot path for NVIDIA B200 (sm_100a).
 *
 * METok ("Multi-Stage Event-based Token Compression", arXiv 2506.02850) removes
 * visual tokens of a long video in three places: after the vision encoder
 * (event segmentation + event-aware reduction, section 3.2.1 and Algorithm 1),
 * inside LLM prefill (hierarchical pruning by text->visual attention and event
 * importance, section 3.2.2, Eq. 6 and 7) and in the decode-time KV cache
 * (section 3.3).  This library is the data-parallel part of that pipeline; the
 * vision tower, text encoder and LLM layers belong to the caller.
 *
 * Conventions shared by every entry point
 *   - Return value: METOK_OK or a negative METOK_ERR_* code.  Nothing throws,
 *     aborts or prints.  Arguments are validated on the host before anything is
 *     launched; a call that fails validation launches nothing.
 *   - Pointers named in the argument comments as DEVICE point to memory of the
 *     current CUDA device, owned by the caller, 16-byte aligned, row-major and
 *     contiguous.  HOST pointers are ordinary host memory read during the call.
 *   - The library never allocates device memory.
 *     Scratch comes from a caller workspace `ws` of at least
 *     metok_*_workspace_bytes(...) bytes (pure host functions).  Its contents
 *     are undefined afterwards; two calls that overlap on the GPU must not
 *     share a workspace.
 *   - Work is enqueued on `stream` (a cudaStream_t passed as void*; NULL is the
 *     legacy default stream) and the call returns without synchronising.
 *     Outputs, including device-resident counts, are valid once the caller has
 *     synchronised with the stream.
 *   - Inputs are never written, except the K/V buffers of metok_kv_compact.
 *   - dtype: METOK_F32 (float) or METOK_BF16 (bfloat16).  bf16 paths accumulate
 *     in fp32; selections compare fp32 scores; ties always go to the lower index.
 *   - Ratios are doubles; every count derived from a ratio is
 *     ceil(ratio * population - 1e-9) evaluated in double.
 *   - Token index j = f*N + p for frame f and position p.
 */
#ifndef METOK_H_
#define METOK_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define METOK_API __attribute__((visibility("default")))
#else
#define METOK_API
#endif

#define METOK_OK               0
#define METOK_ERR_INVALID_ARG (-1)  /* null pointer, size out of range, bad ratio, misaligned pointer */
#define METOK_ERR_UNSUPPORTED (-2)  /* well-formed, but outside the compiled shapes / dtypes */
#define METOK_ERR_WORKSPACE   (-3)  /* ws is NULL or smaller than *_workspace_bytes */
#define METOK_ERR_CUDA        (-4)  /* a launch or driver call failed; see metok_last_cuda_error */
#define METOK_ERR_TIMEOUT     (-5)  /* a bounded device-side wait gave up (reported via status words) */
#define METOK_ERR_TOO_LARGE   (-6)  /* the problem exceeds a fixed built-in capacity (see *_static) */

#define METOK_F32  0
#define METOK_BF16 1

#define METOK_SIM_FLATTEN  0   /* Frobenius inner product of the N x d frame matrices */
#define METOK_SIM_MEANPOOL 1   /* average the N tokens first, then cosine in R^d      */

#define METOK_AGG_MEAN 0       /* event score = mean of its frame scores (section 3.2.1, body text) */
#define METOK_AGG_MAX  1       /* event score = max of its frame scores (Algorithm 1)               */

#define METOK_MODE_TOPK_MERGE 0  /* per-event key-token top-k + merge of the rest      */
#define METOK_MODE_POOL       1  /* Algorithm 1: key frames + adaptive 2-D pooling     */

#define METOK_KV_PAPER 0       /* section 3.3: drop every visual position from layer l1 on */
#define METOK_KV_TOPK  1       /* keep the ceil(ratio*n_vis) best-scored visual tokens per layer */
#define METOK_KV_GIVEN 2       /* the caller supplies the keep lists */

#define METOK_MAX_GROUPS 64

/* ------------------------------------------------------------------------- *
 * (1) Temporal event segmentation -- Eq. 4 and the paragraph after it;
 *     Algorithm 1, "Event temporal segmentation".
 *
 *   sims[i] = cos(v_i, v_{i+1}),  i = 0 .. T-2   (T-1 adjacent pairs)
 *   boundaries = the k-1 smallest sims (lower i first on ties), ascending;
 *                boundary b splits between frame b and b+1
 *   event_offsets = [0, b_1+1, ..., T]  (CSR over frames, k+1 entries)
 *   frame_event[f] = event of frame f
 *
 *   feats        DEVICE [T][N][d] of `dtype`              (input)
 *   sims         DEVICE float [max(T-1,1)]                (output)
 *   boundaries   DEVICE int32 [max(k-1,1)]                (output)
 *   event_offsets DEVICE int32 [k+1]                      (output)
 *   frame_event  DEVICE int32 [T]                         (output)
 *
 *   Norms are clamped below by 1e-8.  There is no minimum event length.
 *   Errors: INVALID_ARG for null/misaligned pointers, T,N,d < 1, k < 1, k > T,
 *   unknown sim_mode or dtype; UNSUPPORTED if d*sizeof(elem) is not a multiple
 *   of 16 or T > 8192; WORKSPACE if ws is too small.
 * ------------------------------------------------------------------------- */
METOK_API size_t metok_segment_events_workspace_bytes(int dtype, int T, int N, int d, int sim_mode);
METOK_API int metok_segment_events(const void* feats, int dtype, int T, int N, int d, int k, int sim_mode,
                         float* sims, int32_t* boundaries, int32_t* event_offsets,
                         int32_t* frame_event, void* ws, size_t ws_bytes, void* stream);

/* ------------------------------------------------------------------------- *
 * (1b) metok_segment_events without any workspace.  The paper has no counterpart
 *      to this entry point; it exists for callers that cannot allocate.
 *
 *   Some hosts of this library may not call cudaMalloc at the point where they
 *   need the segmentation: code running inside a memory pool whose budget is
 *   already fixed, a plugin whose host application owns every allocation, a
 *   real-time loop in which an allocation (an implicit device synchronisation)
 *   is not acceptable.  For them this variant keeps its scratch -- the per-slab
 *   partial sums of the similarity pass -- in a fixed 1 MiB array that is part of
 *   the library image: every GPU that loads the library holds that 1 MiB until
 *   the process exits.  Inputs and outputs are still the caller's.  It computes
 *   exactly what metok_segment_events computes, with the same kernels, and never
 *   calls cudaMalloc, cudaFree or any allocating routine.
 *
 *   Limits and rules
 *   - The problem must fit: metok_segment_events_workspace_bytes(dtype,T,N,d,
 *     sim_mode) <= metok_segment_events_static_capacity() (1 MiB; e.g. FLATTEN with
 *     T*ceil(N*d*elem/16384) <= 131072 -- the 128-frame workload needs 63 KiB).
 *     Larger problems return METOK_ERR_TOO_LARGE and launch nothing.
 *   - The first call on each device looks up the array's device address (a
 *     driver query, no allocation).  Make that first call outside any CUDA
 *     stream capture: while `stream` is being captured such a first call returns
 *     METOK_ERR_UNSUPPORTED and does nothing.  Later calls only launch kernels.
 *   - All calls on one device share the one array.  Nothing in it has to start at
 *     zero (each call overwrites every entry it later reads), but two calls that
 *     overlap on the GPU -- different streams, or one stream per thread -- race
 *     on it and give wrong results.  Serialise them on one stream, or use
 *     metok_segment_events with separate workspaces.
 *   Arguments and the other errors are those of metok_segment_events.
 * ------------------------------------------------------------------------- */
METOK_API size_t metok_segment_events_static_capacity(void);
METOK_API int metok_segment_events_static(const void* feats, int dtype, int T, int N, int d, int k, int sim_mode,
                                float* sims, int32_t* boundaries, int32_t* event_offsets,
                                int32_t* frame_event, void* stream);

/* ------------------------------------------------------------------------- *
 * (1c) Segmentation and the token relevance of Eq. 5 in one pass -- Eq. 4 and
 *      Eq. 5; Algorithm 1, "Event temporal segmentation" and "Key visual-text
 *      semantic identification".
 *
 *   Both need one read of V each and nothing of each other; when the text
 *   embedding is already known at segmentation time this call computes
 *   everything metok_segment_events computes (sim_mode FLATTEN) and, from the same
 *   pass over V,
 *     token_score[j]    = cos(x_j, t)            (what metok_compress_vision's first step computes)
 *     token_inv_norm[j] = 1 / max(|x_j|, 1e-8)
 *   Hand both to metok_compress_vision (token_score argument; params.token_inv_norm)
 *   and it skips its own pass over V.
 *
 *   text_emb       DEVICE [d] of `dtype`                  (input)
 *   token_score    DEVICE float [T*N]                     (output)
 *   token_inv_norm DEVICE float [T*N]                     (output)
 *   the other arguments and errors as in metok_segment_events; UNSUPPORTED also for
 *   rows of more than 8 KiB (use the two separate calls).
 * ------------------------------------------------------------------------- */
METOK_API size_t metok_segment_score_events_workspace_bytes(int dtype, int T, int N, int d);
METOK_API int metok_segment_score_events(const void* feats, int dtype, int T, int N, int d, int k,
                               const void* text_emb, float* sims, int32_t* boundaries,
                               int32_t* event_offsets, int32_t* frame_event, float* token_score,
                               float* token_inv_norm, void* ws, size_t ws_bytes, void* stream);

/* ------------------------------------------------------------------------- *
 * (2) Event-aware token reduction after the vision encoder -- Eq. 5 and
 *     section 3.2.1 ("Key Visual-Text Semantic Identification", "Adaptive
 *     Pooling Strategy"); Algorithm 1.
 *
 *   token_score[j] = cos(x_j, t)                       (Eq. 5, read per token)
 *   frame_score[f] = mean of its N token scores
 *   event_score[e] = mean (or max) of its frame scores
 *   event_is_key   = the ceil(alpha*k) best events
 *
 *   mode TOPK_MERGE: in event e with m_e tokens the
 *     k_e = min(m_e, max(1, ceil(keep*m_e))) best-scored tokens are key tokens
 *     (keep = keep_key for key events, keep_nonkey otherwise); every other token
 *     of the event joins the key token of the same event with which it has the
 *     highest cosine similarity; output token = plain mean, in feature space, of
 *     a key token and the tokens that joined it.  Outputs are ordered by the
 *     key token's index.
 *   mode POOL (Algorithm 1): per event the ceil(beta*len) best-scored frames are
 *     key frames; every frame's G x G token grid (G*G = N) is average-pooled with
 *     window = stride = s1 / s2 (key / other frames of key events) or
 *     s1_nonkey / s2_nonkey (non-key events); edge windows average the cells
 *     that exist; pooled frames are appended in temporal order.
 *
 *   feats         DEVICE [T][N][d]                       (input)
 *   event_offsets DEVICE int32 [k+1] (from metok_segment_events)  (input)
 *   text_emb      DEVICE [d] of `dtype`                  (input)
 *   p             HOST   parameters                      (input)
 *   out_feats     DEVICE [cap][d] of `dtype`             (output; rows >= *n_out untouched)
 *   out_src       DEVICE int32 [cap]  TOPK_MERGE: index of the key token;
 *                                     POOL: index of the window's first token
 *   out_event     DEVICE int32 [cap]  event of the output token
 *   out_members   DEVICE int32 [cap]  number of input tokens averaged (>= 1)
 *   assign        DEVICE int32 [T*N]  output row that each input token went into
 *   token_score   DEVICE float [T*N] (input instead when p->token_inv_norm is set);
 *   frame_score   DEVICE float [T];
 *   event_score   DEVICE float [k];   event_is_key DEVICE uint8 [k]
 *   n_out         DEVICE int32 scalar: number of output tokens
 *   cap           rows available in the out_* arrays; must be at least
 *                 metok_compress_vision_bound(T, N, k, p)
 *
 *   Errors: INVALID_ARG (null/misaligned pointers, sizes < 1, k > T, alpha/keep/
 *   beta outside (0,1], strides < 1, N not a square in POOL mode, cap too small);
 *   UNSUPPORTED (row bytes not a multiple of 16); WORKSPACE.
 * ------------------------------------------------------------------------- */
typedef struct metok_vision_params {
    double alpha;        /* key-event ratio, (0,1]                              */
    int    event_agg;    /* METOK_AGG_*                                         */
    int    mode;         /* METOK_MODE_*                                        */
    double keep_key;     /* TOPK_MERGE: key-token ratio in key events, (0,1]    */
    double keep_nonkey;  /* TOPK_MERGE: key-token ratio in non-key events       */
    double beta;         /* POOL: key-frame ratio, (0,1]                        */
    int    s1, s2;       /* POOL: strides of key / other frames in key events   */
    int    s1_nonkey, s2_nonkey;  /* POOL: the same for non-key events (the paper: s/alpha) */
    const float* token_inv_norm;  /* NULL, or DEVICE float [T*N] from metok_segment_score_events: then the
                                     token_score argument is an INPUT and the Eq. 5 pass over V is skipped */
    const uint8_t* key_events_given;  /* NULL, or DEVICE uint8 [k]: the key events are the caller's (non-zero =
                                         key) instead of the ceil(alpha*k) best-scored ones -- the ablation
                                         with randomly chosen key events; event_is_key returns them */
    const uint8_t* key_frames_given;  /* POOL: NULL, or DEVICE uint8 [T]: the key frames are the caller's (non-zero =
                                         key) instead of the ceil(beta*|E_j|) best-scored frames of every
                                         event -- the ablation with randomly chosen key frames */
} metok_vision_params;

METOK_API int    metok_compress_vision_bound(int T, int N, int k, const metok_vision_params* p);
METOK_API size_t metok_compress_vision_workspace_bytes(int dtype, int T, int N, int d, int k, int cap,
                                             const metok_vision_params* p);
METOK_API int metok_compress_vision(const void* feats, int dtype, int T, int N, int d,
                          const int32_t* event_offsets, int k, const void* text_emb,
                          const metok_vision_params* p,
                          void* out_feats, int32_t* out_src, int32_t* out_event,
                          int32_t* out_members, int32_t* assign, float* token_score,
                          float* frame_score, float* event_score, uint8_t* event_is_key,
                          int32_t* n_out, int cap, void* ws, size_t ws_bytes, void* stream);

/* ------------------------------------------------------------------------- *
 * (3) One level of hierarchical token pruning during prefill -- section 3.2.2,
 *     Eq. 6 and 7; attention form and scale of Eq. 2.
 *
 *   The sequence has S positions; the visual tokens occupy
 *   [vis_start, vis_start + n_vis), the Lt text queries are the LAST Lt positions.
 *   scores[j] = mean over all Hq heads h and Lt text queries q of
 *               softmax_u( Q[h][q] . K[g(h)][u] * softmax_scale )[vis_start + j],
 *   the softmax taken over the keys query q may see, u <= S - Lt + q (causal);
 *   g(h) = h / (Hq / Hkv).
 *   Visual token j has a class token_group[j] in [0, G).  In class g the
 *   min(population, group_budget[g]) best-scored tokens survive; every
 *   non-visual position survives.  keep_idx lists the surviving positions in
 *   ascending order, *S_out is their number, and
 *   hidden_out[i] = hidden[keep_idx[i]].
 *
 *   q_text       DEVICE [Hq][Lt][dh]        k_all  DEVICE [Hkv][S][dh]
 *   hidden       DEVICE [S][D]              (may be NULL with hidden_out NULL: no gather)
 *   token_group  DEVICE int32 [n_vis]
 *   group_budget HOST   int32 [G]  (from metok_retention_budgets, or any counts >= 0;
 *                                   a budget above the population is clamped)
 *   scores       DEVICE float [n_vis]       keep_idx DEVICE int32 [S]
 *   S_out        DEVICE int32 scalar        hidden_out DEVICE [S][D] capacity
 *
 *   Errors: INVALID_ARG (null/misaligned, sizes < 1, Hq % Hkv != 0, Lt > S,
 *   visual span outside [0, S-Lt], G outside [1, METOK_MAX_GROUPS], negative
 *   budget); UNSUPPORTED (dh not in {64,128} for bf16, dh > 128 or dh % 4 for f32,
 *   D*sizeof(elem) % 16 != 0); WORKSPACE.
 * ------------------------------------------------------------------------- */
METOK_API size_t metok_prefill_prune_workspace_bytes(int dtype, int Hq, int Hkv, int Lt, int S, int dh, int n_vis);
METOK_API int metok_prefill_prune(const void* q_text, const void* k_all, const void* hidden, int dtype,
                        int Hq, int Hkv, int Lt, int S, int dh, int D, int vis_start, int n_vis,
                        const int32_t* token_group, int G, const int32_t* group_budget,
                        float softmax_scale, float* scores, int32_t* keep_idx, int32_t* S_out,
                        void* hidden_out, void* ws, size_t ws_bytes, void* stream);

/* The two halves of metok_prefill_prune as calls of their own, for a caller that shards the
 * attention heads over several GPUs (each rank: its own query heads and the KV heads they use,
 * whole groups) and adds the ranks' scores before selecting:
 *   metok_attention_scores: scores[j] = (sum over THIS call's heads h and the Lt text queries q of
 *     softmax(...)[vis_start + j]) / rows_total, rows_total = all ranks' Hq * Lt (0: this call's),
 *     so that the sum of the ranks' scores is metok_prefill_prune's score.  Arguments, layouts,
 *     errors and workspace size as metok_prefill_prune; rows_total < Hq*Lt (and != 0) is INVALID_ARG.
 *   metok_prune_by_scores: the class-wise top-k and the hidden-state gather of
 *     metok_prefill_prune on the caller's DEVICE scores[n_vis]; the visual span may lie anywhere
 *     in [0, S].  Workspace: metok_prune_by_scores_workspace_bytes(). */
METOK_API int metok_attention_scores(const void* q_text, const void* k_all, int dtype, int Hq, int Hkv, int Lt,
                        int S, int dh, int vis_start, int n_vis, float softmax_scale, int rows_total,
                        float* scores, void* ws, size_t ws_bytes, void* stream);
METOK_API size_t metok_prune_by_scores_workspace_bytes(void);
METOK_API int metok_prune_by_scores(const float* scores, const void* hidden, int dtype, int S, int D,
                        int vis_start, int n_vis, const int32_t* token_group, int G,
                        const int32_t* group_budget, int32_t* keep_idx, int32_t* S_out, void* hidden_out,
                        void* ws, size_t ws_bytes, void* stream);

/* Eq. 6 and 7: token budgets after pruning level `stage` (1, 2, 3 = layers l1,
 * l2, l3; 0 = before l1) for N0 = {key-event tokens, non-key-event tokens}
 * first passed into the LLM:  R_key = 1, r, r^2, 0 ;  R_nonkey = 1, alpha*r, 0, 0.
 * (The equations leave l = l3 and l = l2 unassigned; both take the next case.)
 * HOST pointers.  budget[g] = min(N0[g], ceil(R_g * N0[g] - 1e-9)). */
METOK_API int metok_retention_budgets(double alpha, double r, int stage, const int32_t* N0, int32_t* budget);

/* ------------------------------------------------------------------------- *
 * (3b) The pruning levels l1, l2, l3 in one call -- section 3.2.2, Eq. 6 and 7.
 *
 *   Level s (1-based) is metok_prefill_prune on the tokens that survived level
 *   s-1, with the budgets of metok_retention_budgets(alpha, r, s, N0); a
 *   survivor keeps its class.  Everything is enqueued on `stream`; nothing is
 *   read back between levels.  N0 = {key-event, non-key-event} counts of the
 *   first level's token_group (classes 0 and 1; HOST): they fix the sizes of all
 *   levels, n_vis_s = budget_0(s-1) + budget_1(s-1) (n_vis_1 = N0[0] + N0[1]),
 *   S_s = S - n_vis + n_vis_s, which metok_prune_schedule_sizes returns.
 *
 *   Per level s, all DEVICE: q_text [Hq][Lt][dh] and k_all [Hkv][S_s][dh] of that
 *   layer (rows of the survivors, in order), hidden [S_s][D] / hidden_out
 *   (both or neither), scores [n_vis_s], keep_idx [S_s], S_out scalar,
 *   token_group [n_vis_s] (level 1: input; later levels: written), origin
 *   [n_vis_s] (written: index among the first level's visual tokens).
 *   `status` DEVICE int32: written 0, or METOK_ERR_INVALID_ARG when N0 does not
 *   match the first level's classes (later levels are then meaningless).
 *
 *   Errors: those of metok_prefill_prune per level; INVALID_ARG also for
 *   n_levels outside [1, 3], N0 not summing to n_vis, or a level without visual
 *   tokens.  Workspace: the largest of the levels' (..._schedule_workspace_bytes; 0 = invalid).
 * ------------------------------------------------------------------------- */
typedef struct {
    const void* q_text;
    const void* k_all;
    const void* hidden;
    void* hidden_out;
    float* scores;
    int32_t* keep_idx;
    int32_t* S_out;
    int32_t* token_group;
    int32_t* origin;
} metok_prune_level;

/* HOST: n_vis_of_level[s] for s = 0..n_levels (entry n_levels = survivors of the last level). */
METOK_API int metok_prune_schedule_sizes(int n_levels, double alpha, double r, const int32_t* N0,
                        int32_t* n_vis_of_level);
METOK_API size_t metok_prefill_prune_schedule_workspace_bytes(int n_levels, int dtype, int Hq, int Hkv, int Lt,
                        int S, int dh, int n_vis, double alpha, double r, const int32_t* N0);
METOK_API int metok_prefill_prune_schedule(const metok_prune_level* levels, int n_levels, int dtype,
                        int Hq, int Hkv, int Lt, int S, int dh, int D, int vis_start, int n_vis,
                        double alpha, double r, const int32_t* N0, float softmax_scale,
                        int32_t* status, void* ws, size_t ws_bytes, void* stream);

/* The K/V keep lists that follow from the recorded keep lists of the levels (section 3.3: the cache
 * is pruned in line with the hierarchical pruning).  Layer l lies in group g = number of pruning
 * layers level_layer[s] <= l; its cache holds the rows of level g's input (all of them for g = 0),
 * S - n_vis + n_vis_of_level[g] rows, and keeps what level g + 1 kept; layers at or beyond the last
 * pruning layer keep all their rows.  Call it on the stream of metok_prefill_prune_schedule after
 * that call; the lists are in the form policy GIVEN of metok_kv_compact takes (one call per group
 * of layers, whose caches have the same length).
 *   level_layer  HOST int32 [n_levels]: the pruning layers l1 < l2 < l3 (0-based)
 *   kv_keep_idx  DEVICE int32 [L][S] (row stride S); kv_keep_len DEVICE int32 [L]
 *   kv_S_cur     HOST int32 [L] (output): rows of layer l's cache before compaction
 *   ws           DEVICE, at least 4*L bytes
 * Errors: INVALID_ARG (null pointers, layers not ascending, N0 not summing to n_vis);
 * UNSUPPORTED (L > 1024); WORKSPACE. */
METOK_API int metok_prune_schedule_kv_lists(const metok_prune_level* levels, int n_levels,
                        const int32_t* level_layer, int L, int S, int n_vis, double alpha, double r,
                        const int32_t* N0, int32_t* kv_keep_idx, int32_t* kv_keep_len, int32_t* kv_S_cur,
                        void* ws, size_t ws_bytes, void* stream);

/* ------------------------------------------------------------------------- *
 * (4) KV-cache selection and in-place compaction -- section 3.3.
 *
 *   For every layer l a keep list (ascending positions < S_cur) is chosen:
 *     PAPER: layers l < l1 keep everything; layers l >= l1 drop all visual
 *            positions [vis_start, vis_start+n_vis) (0-based layers);
 *     TOPK : keep the ceil(keep_ratio*n_vis) best-scored visual tokens and all
 *            non-visual positions (scores shared by all layers, or one row per layer);
 *     GIVEN: keep_idx / keep_len are inputs.
 *   Then, for K and V of every layer and every head h,
 *     X[l][h][i][:] = X[l][h][keep_idx[l][i]][:]   for i < keep_len[l], in place;
 *   rows at and beyond the new length are unspecified afterwards.
 *
 *   k_layers, v_layers HOST arrays of L DEVICE pointers, each [Hkv][S_cap][dh]
 *   scores    DEVICE float [n_vis] or [L][n_vis] (TOPK), else NULL
 *   keep_idx  DEVICE int32 [L][S_cur]; keep_len DEVICE int32 [L]
 *             (outputs for PAPER / TOPK, inputs for GIVEN)
 *   new_len   DEVICE int32 [L] (output; equals keep_len)
 *
 *   GIVEN lists are checked on the device before any row is indexed through them
 *   (0 <= keep_len[l] <= S_cur, entries strictly ascending inside [0, S_cur)).  A
 *   layer whose list fails is left untouched, reports new_len[l] = S_cur, and the
 *   device status word (first int32 of ws, valid after the stream is synchronised)
 *   reads METOK_ERR_INVALID_ARG; the other layers are compacted as usual.  The
 *   status word reads METOK_OK otherwise.
 *   Errors: INVALID_ARG (null/misaligned, sizes < 1, S_cur > S_cap, span outside
 *   [0,S_cur], ratio outside [0,1], l1 < 0, unknown policy); UNSUPPORTED
 *   (dh*sizeof(elem) % 16 != 0); WORKSPACE.
 * ------------------------------------------------------------------------- */
METOK_API size_t metok_kv_compact_workspace_bytes(int dtype, int L, int Hkv, int S_cur, int dh, int policy, int n_vis);
METOK_API int metok_kv_compact(void* const* k_layers, void* const* v_layers, int dtype, int L, int Hkv,
                     int S_cap, int S_cur, int dh, int policy, int l1, double keep_ratio,
                     int vis_start, int n_vis, const float* scores, int scores_per_layer,
                     int32_t* keep_idx, int32_t* keep_len, int32_t* new_len,
                     void* ws, size_t ws_bytes, void* stream);

/* ------------------------------------------------------------------------- *
 * helpers (host only, no CUDA work)
 * ------------------------------------------------------------------------- */
/* Per-kernel timing for benchmarks.  Between metok_profile_begin() and
 * metok_profile_end() every kernel the library launches is bracketed by CUDA
 * events on the launching stream.  metok_profile_end synchronises with those
 * events and writes one text line per kernel name, "name launches total_ms\n",
 * in first-launch order, into `out` (HOST, `cap` bytes, NUL-terminated; truncated
 * if too small).  Returns the number of kernel launches recorded, or a negative
 * status.  Not thread-safe against concurrent calls into the library; adds two
 * event records per launch, so never leave it on outside a measurement.
 * Calls made while their stream is being captured into a CUDA graph put the
 * brackets into the graph as event-record nodes: every replay of the graph then
 * times its kernels without the host's launch gaps.  metok_profile_read stops
 * bracketing further launches and reports like metok_profile_end but keeps the
 * events, so that the graph can be replayed and read again; metok_profile_end
 * releases them (destroy the graph first).  metok_profile_scope(label) names the
 * brackets recorded from then on (label without blanks or '/', NULL or "" for none):
 * they are reported as "label/name", so that launches of one kernel made for different
 * steps of the path can be told apart.  The paper has no counterpart of these calls. */
METOK_API int metok_profile_begin(void);
METOK_API int metok_profile_scope(const char* label);
METOK_API int metok_profile_read(char* out, size_t cap);
METOK_API int metok_profile_end(char* out, size_t cap);

/* Debug builds (lib/libmetok_debug.so: compiled with METOK_DEBUG_SHORT_WAIT and METOK_DEBUG_BOUNDS).
 * There the bounded device-side waits give up after a few thousand polls, every data-dependent
 * row or slot index is range-checked (a bad one is counted in int32 word 2 of the workspace and
 * replaced by 0: nothing traps or faults), and metok_debug_set(METOK_DEBUG_WITHHOLD_COPY, mask)
 * makes the producer of the kernels named in `mask` skip one copy in the calls made from then on,
 * so that the waiting side runs into its limit, the CTA unwinds (copies drained, tensor memory
 * freed) and the call's status word -- int32 word 0 of the workspace -- reads METOK_ERR_TIMEOUT.
 * mask bits: 1 merge-assign, 2 attention statistics, 4 attention column sums, 8 averaging,
 * 16 hidden-row gather; 0 switches it off.  metok_debug_build() returns 1 | 2 for such a build and
 * 0 for the normal library, in which metok_debug_set returns METOK_ERR_UNSUPPORTED and does
 * nothing.  The paper has no counterpart of these two calls. */
#define METOK_DEBUG_WITHHOLD_COPY 1
METOK_API int metok_debug_set(int what, int value);
METOK_API int metok_debug_build(void);

METOK_API const char* metok_status_string(int status);
METOK_API int metok_last_cuda_error(void);   /* cudaError_t of the last METOK_ERR_CUDA on this thread, else 0 */
METOK_API int metok_version(void);           /* major*10000 + minor*100 + patch */

#ifdef __cplusplus
}
#endif
#endif /* METOK_H_ */
