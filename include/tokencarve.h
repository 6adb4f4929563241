/*
 * tokencarve.h -- C ABI of the IPGS carve library (TokenCarve, Sec. 3.3).
 *
 * The library runs the two-stage Information-Preservation-Guided Selection that TokenCarve
 * applies once per request at prefill, between LLM layers 2 and 3:
 *
 *   Stage I  (Sec. 3.3.1)  score every visual token  E(x) = (1-lambda) C(x) + lambda S(x)
 *                          (Eq. 3-8), C from the SVD of the attention-output matrix (Eq. 3-5,
 *                          3-6), S the mean attention the token receives (Eq. 3-7); keep the
 *                          L_vc (1 + rho) best.
 *   Stage II (Sec. 3.3.2)  split the survivors by score into Set A / Set B (Eq. 3-9), match
 *                          every Set-B token to its most cosine-similar Set-A token
 *                          (Eq. 3-10), merge the L_vc * rho best-matched Set-B tokens into
 *                          their match by a plain average, keep the rest; L_vc tokens result,
 *                          in their original order (Sec. 5).
 *
 * Conventions for every entry point
 *   - Every data pointer is DEVICE memory owned by the caller (the *_host entry point is the
 *     one exception and says so), contiguous, row-major, 16-byte aligned.  The library
 *     allocates nothing: all scratch is carved out of the caller's workspace `ws`, whose
 *     size tc_workspace_bytes() reports for a given tc_params.
 *   - Layouts:  O, X [B, N, d];  A [B, H, T, N];  K, V [B, H, N, dh];
 *     outputs   Xo [B, keep, d];  Ko, Vo [B, H, keep, dh];  kept_idx [B, keep].
 *     Element type is tc_params.dtype for O, A, X, K, V and the outputs; scores, singular
 *     values and similarities are float32; indices are int32 token numbers in [0, N).
 *   - Calls only enqueue work on `stream` and never synchronise.  Errors the host can see
 *     (bad sizes, NULL pointers, short workspace) return a status immediately and enqueue
 *     nothing.  Conditions only the device can see are written per image to `img_status`
 *     (TC_OK when fine) and never trap; they are valid once the stream has been synchronised.
 *   - Index lists are in ascending token order.  Every tie (equal scores, equal
 *     similarities) goes to the lower token index.
 *   - Index lists a caller hands in (setA, setB, kept_idx, merge_src, merge_dst of the staged
 *     calls) are checked on the device: a token number outside [0, N) is never used as an
 *     address; the entry is skipped (a kept row becomes zeros, a merge source is left out, a
 *     match is dropped) and TC_ERR_INVALID_ARG is recorded for that image, to be read with
 *     tc_stage_status().  Numbers inside the range are taken as given.
 *   - The first tc_score / tc_carve / tc_carve_host on a device creates the library's internal
 *     streams and events (image groups, copy streams): make that first call outside any stream
 *     capture.  Later calls create nothing and can be captured into a CUDA graph.
 */
#ifndef TOKENCARVE_H
#define TOKENCARVE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  TC_OK = 0,
  TC_ERR_INVALID_ARG = 1,   /* NULL pointer, size or parameter out of range                 */
  TC_ERR_UNSUPPORTED = 2,   /* shape outside what the kernels handle                         */
  TC_ERR_WORKSPACE = 3,     /* ws_bytes smaller than tc_workspace_bytes()                    */
  TC_ERR_NOT_CONVERGED = 4, /* img_status: Jacobi hit max_sweeps before its tolerance        */
  TC_ERR_CUDA = 5,          /* a CUDA runtime call failed                                    */
  TC_ERR_RANK_CAP = 6,      /* img_status: numerical rank reached rank_cap; rerun that image
                               with a larger rank_cap or with rank_cap = 0                   */
  TC_ERR_BREAKDOWN = 7,     /* img_status: a Cholesky pivot was not positive                 */
  TC_ERR_SCRATCH_LIMIT = 8  /* tc_attn_score_noalloc: request larger than its built-in scratch */
} tc_status;

typedef enum { TC_F16 = 0, TC_F32 = 1, TC_BF16 = 2 } tc_dtype;

/* tc_params.flags: variants kept beside the paper's own choices (0 = the paper's).
 *   Eq. 3-10 matches on the rows of the attention output O.  TC_FLAG_SIM_X matches on the
 *   hidden states X instead, TC_FLAG_SIM_MEAN_K on the mean over the heads of K (the features
 *   ToMe, which Sec. 3.3.2 takes its merging from, matches on).
 *   Sec. 3.3.2 merges with ToMe's plain average.  TC_FLAG_WEIGHTED_MERGE weights every token of
 *   a merged group with its IPGS score E (Eq. 3-8); a group whose scores do not add up to a
 *   positive number falls back to the plain average. */
#define TC_FLAG_SIM_O 0u
#define TC_FLAG_SIM_X 1u
#define TC_FLAG_SIM_MEAN_K 2u
#define TC_FLAG_SIM_MASK 3u
#define TC_FLAG_WEIGHTED_MERGE 16u

/* How Eq. 3-8 combines the two terms: on the raw C and S (the equation as printed), or on
 * C / sum(C) and S / sum(S) so that both terms have the same scale. */
typedef enum { TC_NORM_NONE = 0, TC_NORM_SUM1 = 1 } tc_score_norm;

typedef struct tc_params {
  int32_t batch;      /* B   images                                                          */
  int32_t n_tokens;   /* N = L_v  visual tokens per image                                    */
  int32_t d_model;    /* d   width of O and X                                                */
  int32_t n_heads;    /* H                                                                   */
  int32_t head_dim;   /* dh                                                                  */
  int32_t n_query;    /* T   query rows in the attention slice A                             */
  int32_t keep;       /* L_vc, 1..N                                                          */
  int32_t n_merge;    /* M;  -1 => floor(keep * rho), clamped to [0, N - keep]               */
  float   rho;        /* merge proportion of Sec. 3.3.1/3.3.2, in [0, 1]                     */
  float   lambda;     /* weight of Eq. 3-8, in [0, 1]                                        */
  float   rank_tol;   /* r of Eq. 3-5/3-6 = #{ sigma_i > rank_tol * sigma_1 }; 0 => all      */
  int32_t dtype;      /* tc_dtype of O, A, X, K, V and of Xo, Ko, Vo                         */
  int32_t score_norm; /* tc_score_norm                                                       */
  int32_t max_sweeps; /* bound on Jacobi sweeps (<= 0 => 30)                                 */
  int32_t rank_cap;   /* 0 => full N x N eigen-decomposition of the Gram matrix.
                         k > 0 (k < N) => the caller states that the numerical rank r is
                         below k: only a k-dimensional dominant subspace is decomposed.  The
                         device checks r <= k - 8 and reports TC_ERR_RANK_CAP otherwise.
                         Singular values beyond the k-th are then reported as 0.             */
  uint32_t flags;     /* TC_FLAG_* variants, 0 = the paper's choices                         */
} tc_params;

/* Counts derived from the parameters (Sec. 3.3.1 last paragraph, Eq. 3-9):
 * M merged tokens, P = keep + M Stage-I survivors, nA = floor(P / 2), nB = P - nA. */
tc_status tc_counts(const tc_params* p, int32_t* M, int32_t* P, int32_t* nA, int32_t* nB);

/* Bytes of device workspace any of the calls below needs for these parameters. */
tc_status tc_workspace_bytes(const tc_params* p, size_t* bytes);

/*
 * Stage I scores (Sec. 3.3.1, Eq. 3-5 ... 3-8).
 *   O [B,N,d], A [B,H,T,N] in;  E [B,N] out (required);
 *   optional outs (NULL to skip): C [B,N] Eq. 3-6, S [B,N] Eq. 3-7,
 *   sigma [B, min(N,d)] singular values, descending, rank [B] the r used in Eq. 3-6.
 *   img_status [B] int32 (required).
 */
tc_status tc_score(const tc_params* p, const void* O, const void* A, float* E, float* C,
                   float* S, float* sigma, int32_t* rank, int32_t* img_status, void* ws,
                   size_t ws_bytes, void* stream);

/*
 * Stage I prune and the Set A / Set B split (Sec. 3.3.1 last paragraph, Eq. 3-9).
 *   E [B,N] in;  setA [B,nA], setB [B,nB] out: Set A holds the nA best-scored tokens, Set B
 *   the next nB; each list in ascending token index.
 */
tc_status tc_prune(const tc_params* p, const float* E, int32_t* setA, int32_t* setB, void* ws,
                   size_t ws_bytes, void* stream);

/*
 * Stage II matching (Eq. 3-10 and the paragraph after it).
 *   O [B,N,d], setA, setB in.  Cosine similarity of the L2-normalised rows of O between every
 *   Set-B and Set-A token; each Set-B token's best Set-A match; the M Set-B tokens with the
 *   highest best-similarity are merged.  The call matches on the rows of whatever [B,N,d]
 *   matrix it is given (pass X with TC_FLAG_SIM_X); with TC_FLAG_SIM_MEAN_K the argument is
 *   K [B,H,N,dh] and the features are its mean over the heads.
 *   merge_src [B,M] (ascending), merge_dst [B,M] (the match of merge_src[i]),
 *   kept_idx [B,keep] = Set A plus the unmerged Set-B tokens, ascending.
 */
tc_status tc_merge(const tc_params* p, const void* O, const int32_t* setA, const int32_t* setB,
                   int32_t* merge_src, int32_t* merge_dst, int32_t* kept_idx, void* ws,
                   size_t ws_bytes, void* stream);

/*
 * Merge and gather (Sec. 3.3.2 last paragraph: ToMe's average; Sec. 5: original order).
 *   Row j of the output is row kept_idx[j] of the input, or, when that token is a merge
 *   destination, the plain mean of it and all tokens merged into it (float32 accumulate,
 *   one rounding to the storage type).  The same map is applied to X and to every head of
 *   K and V.  K, V, Ko, Vo may all be NULL (then only X is compacted).
 */
tc_status tc_compact(const tc_params* p, const void* X, const void* K, const void* V,
                     const int32_t* kept_idx, const int32_t* merge_src,
                     const int32_t* merge_dst, void* Xo, void* Ko, void* Vo, void* ws,
                     size_t ws_bytes, void* stream);

/* tc_compact with the score-weighted merge (TC_FLAG_WEIGHTED_MERGE as a staged call): E [B,N]
 * float32 (device) are the weights, e.g. tc_score's E.  Everything else as tc_compact. */
tc_status tc_compact_weighted(const tc_params* p, const void* X, const void* K, const void* V,
                              const int32_t* kept_idx, const int32_t* merge_src,
                              const int32_t* merge_dst, const float* E, void* Xo, void* Ko,
                              void* Vo, void* ws, size_t ws_bytes, void* stream);

/*
 * Device-side findings of the last tc_merge or tc_compact that used the workspace `ws` (each of
 * them clears the record when it starts): img_status [B] int32 (device) receives, per image,
 * TC_OK or TC_ERR_INVALID_ARG (a list entry outside [0, N) was skipped).  Enqueued on `stream`
 * behind that call; valid once the stream has been synchronised.  The paper has no counterpart:
 * it is how the staged calls of Sec. 3.3.2 report without a status argument of their own.
 */
tc_status tc_stage_status(const tc_params* p, const void* ws, size_t ws_bytes, int32_t* img_status,
                          void* stream);

/*
 * The whole path (Sec. 3.3): score -> prune -> split -> match -> merge -> gather, one
 * enqueue, no host synchronisation inside.
 */
tc_status tc_carve(const tc_params* p, const void* O, const void* A, const void* X,
                   const void* K, const void* V, void* Xo, void* Ko, void* Vo,
                   int32_t* kept_idx, int32_t* img_status, void* ws, size_t ws_bytes,
                   void* stream);

/*
 * tc_carve for callers whose tensors live in HOST memory (pinned for the copies to be
 * asynchronous).  O, A, X, K, V, Xo, Ko, Vo, kept_idx and img_status are host pointers.  The
 * batch is cut into up to four chunks: the upload of the next chunk and the download of the
 * previous one run on two internal copy streams while the current chunk is carved on `stream`;
 * everything is forked from `stream` and joined back into it, so work enqueued on `stream`
 * afterwards sees the results in host memory once it runs.
 * `ws` is device memory of at least tc_workspace_bytes_host() bytes (staging + scratch).
 */
tc_status tc_workspace_bytes_host(const tc_params* p, size_t* bytes);
tc_status tc_carve_host(const tc_params* p, const void* O, const void* A, const void* X,
                        const void* K, const void* V, void* Xo, void* Ko, void* Vo,
                        int32_t* kept_idx, int32_t* img_status, void* ws, size_t ws_bytes,
                        void* stream);

/*
 * Attention scores without any caller-provided scratch (the paper has no counterpart; the
 * arithmetic is Eq. 3-7, the same kernels tc_score runs for S).
 *
 * Who needs it: code that may not allocate device memory at the point where it wants the
 * scores, and so cannot produce the workspace the other entry points ask for.  Typical cases
 * are a plug-in running inside another framework's forward pass whose memory pool it must not
 * touch, a real-time serving loop where cudaMalloc's implicit device synchronisation is not
 * acceptable, and a process that has handed all of the GPU's memory to a pool at start-up.
 *
 *   A [B,H,T,N] in (device, tc_params.dtype);  S [B,N] float32 out (device).  Only batch,
 *   n_tokens, n_heads, n_query and dtype of `p` matter, but `p` must be valid as a whole.
 *
 * The partial column sums go into a fixed array of TC_NOALLOC_SCRATCH_BYTES that is part of
 * the library image: a GPU holds that much memory from the moment the part of the library that
 * contains the array is loaded onto it (with the CUDA runtime's lazy loading that is this
 * function's first call on the device) until the process exits.  The call needs
 * B * chunks * N floats of it, where chunks = min(64, (H*T)/32, ceil(592/B)) (at least 1);
 * a larger request returns TC_ERR_SCRATCH_LIMIT and enqueues nothing.
 *
 * The first call on each device looks up the array's device address (a host-side runtime
 * query, done with that device current).  That query, and the loading of the code it may
 * trigger, can allocate and synchronise inside the driver: make the first call at start-up,
 * outside any stream capture and outside latency-critical code.  After it, no call of this
 * function allocates or frees memory (it calls neither cudaMalloc nor cudaFree nor any library
 * that does).  `stream` must belong to the device that is current at the call: the address is
 * remembered per current device.  The remembered address is not valid across cudaDeviceReset.
 * All calls on a device share the one array, which keeps whatever the previous call left in
 * it; each call overwrites the part it uses before reading it, so nothing has to be cleared,
 * but two calls that overlap on the GPU (different streams, or different host threads without
 * ordering) race on it.  Order them on one stream.
 */
#define TC_NOALLOC_SCRATCH_BYTES (4u << 20)
tc_status tc_attn_score_noalloc(const tc_params* p, const void* A, float* S, void* stream);

/*
 * The Gram matrix behind the SVD of Sec. 3.3.1 (O O^T = U Sigma^2 U^T) and the similarity of
 * Eq. 3-10, exposed for inspection: G [B,N,N] float32 out.
 */
tc_status tc_gram(const tc_params* p, const void* O, float* G, void* stream);

/*
 * The product kernel of the subspace solve behind Eq. 3-5 / 3-6 (Sec. 3.3.1), exposed for
 * inspection: C [batch][M][NN] = A B^T for float32 A [batch][M][K] and B [batch][NN][K] (device,
 * row-major, 16-byte aligned), computed on the tensor cores with every operand value used as two
 * TF32 numbers (three products per term, float32 accumulation), so that the result is as good
 * as a float32 product.  C and / or CT (the transposed result [batch][NN][M]) are written;
 * either may be NULL, not both.  NN is 128, 144, 160 or 192 and K a multiple of 4, else
 * TC_ERR_UNSUPPORTED.  img_status [batch] (may be NULL) receives TC_ERR_CUDA for an image whose
 * tile pipeline gave up.  Allocates nothing, only enqueues.
 */
tc_status tc_matmul_f32x3(const float* A, const float* B, float* C, float* CT, int32_t batch,
                          int32_t M, int32_t NN, int32_t K, int32_t* img_status, void* stream);

/*
 * Sec. 3.2 ("Visual Token Information") and the appendix "Attention Output Matrix Rank": the
 * information quantity of a set of visual tokens is the matrix rank of their rows of the
 * attention-output matrix, followed as tokens are removed.  For every image b, the singular
 * values of the n_sub x d matrix made of the rows idx[b][0..n_sub) of O and its numerical rank
 * #{sigma_i > rank_tol * sigma_1}, from the same Gram and eigen kernels as tc_score (rank_cap
 * applies as there: 0 = full solve, otherwise a bound on the rank, checked on the device).
 *   p        describes O ([batch, n_tokens, d_model], dtype) and rank_tol, rank_cap, max_sweeps;
 *            keep, n_merge, rho, lambda, score_norm are not used
 *   O        device, [B, N, d]
 *   idx      device, [B, n_sub] int32, distinct token numbers in [0, N) in any order (the
 *            result does not depend on the order); NULL = all rows, n_sub must then be N.  A
 *            number outside [0, N) gives TC_ERR_INVALID_ARG in that image's status, never a fault
 *   sigma    device, [B, min(n_sub, d)] float32 out, descending; may be NULL
 *   rank     device, [B] int32 out
 *   img_status  device, [B] int32 out, as in tc_score
 *   ws       device scratch of tc_rank_workspace_bytes(p, n_sub) bytes, 16-byte aligned, owned by
 *            the caller; nothing is allocated.  Asynchronous on `stream`.
 * Returns TC_ERR_INVALID_ARG / TC_ERR_UNSUPPORTED / TC_ERR_WORKSPACE with nothing enqueued.
 */
tc_status tc_rank_workspace_bytes(const tc_params* p, int32_t n_sub, size_t* bytes);
tc_status tc_rank(const tc_params* p, const void* O, const int32_t* idx, int32_t n_sub,
                  float* sigma, int32_t* rank, int32_t* img_status, void* ws, size_t ws_bytes,
                  void* stream);

/*
 * Sec. 3.1 (the LLM input is the sequence [system tokens, visual tokens, prompt tokens]) and
 * the Conclusion (the surviving tokens keep their original positional relationships: rotary
 * encodings of the later layers use the original position IDs): the hidden-state sequence the
 * layers after the compression run on, and the original position of each of its rows.
 *   p        batch, n_tokens (= the visual tokens before compression), d_model, dtype, keep
 *   n_sys, n_text  numbers of system and prompt tokens (>= 0)
 *   Hs       device, [B, n_sys + n_tokens + n_text, d] hidden states before the compression
 *            (only its system and prompt rows are read; may be NULL when there are none)
 *   Xo       device, [B, keep, d] compacted visual tokens (tc_compact / tc_carve output)
 *   kept_idx device, [B, keep] int32 original visual-token numbers, ascending (same output)
 *   Ho       device, [B, n_sys + keep + n_text, d] out
 *   pos      device, [B, n_sys + keep + n_text] int32 out: 0 .. n_sys-1, n_sys + kept_idx,
 *            n_sys + n_tokens .. (strictly ascending)
 * Row lengths must be whole 16-byte vectors, pointers 16-byte aligned.  No workspace; asynchronous
 * on `stream`.  kept_idx is trusted to lie in [0, n_tokens): it only enters `pos`.
 */
tc_status tc_reassemble(const tc_params* p, int32_t n_sys, int32_t n_text, const void* Hs,
                        const void* Xo, const int32_t* kept_idx, void* Ho, int32_t* pos,
                        void* stream);

/*
 * The layer-2 probe (Sec. 3.1, Eq. 3-1 and 3-2; Sec. 3.2: the visual slice): what the compression
 * reads from the second LLM layer, produced from that layer's queries, keys and values without
 * writing its probability matrix out.  The sequence is [n_sys system, n_tokens visual, n_text
 * prompt] tokens, L = n_sys + n_tokens + n_text.
 *   p        batch, n_tokens, n_heads, head_dim (128), d_model (= n_heads * head_dim), dtype
 *            (TC_F16 or TC_BF16), n_query = the number T of probe rows
 *   Q, K, V  device, [B, H, L, dh], taken as given (rotary encodings already applied)
 *   O        device out, [B, n_tokens, H * dh]: the visual rows of Z = Softmax(Q K^T / sqrt(dh)) V,
 *            heads side by side (tc_score's O); NULL = not wanted (V and ws may then be NULL)
 *   A        device out, [B, H, T, n_tokens]: the attention the rows probe_start .. probe_start +
 *            T - 1 of the sequence pay to the visual tokens (tc_score's A); NULL = not wanted
 *   The attention is causal (row i sees the keys j <= i); a visual token a probe row cannot see
 *   gets probability 0.  float32 scores and sums, probabilities rounded to the storage type
 *   before they multiply V.
 *   img_status [B] as in tc_score.  ws: device scratch of tc_probe_workspace_bytes() bytes (the
 *   transposed V), owned by the caller; nothing is allocated; asynchronous on `stream`.
 * Returns TC_ERR_UNSUPPORTED for float32 storage or head_dim != 128.
 */
tc_status tc_probe_workspace_bytes(const tc_params* p, int32_t n_sys, int32_t n_text, size_t* bytes);
tc_status tc_probe(const tc_params* p, int32_t n_sys, int32_t n_text, int32_t probe_start,
                   const void* Q, const void* K, const void* V, void* O, void* A,
                   int32_t* img_status, void* ws, size_t ws_bytes, void* stream);

/*
 * Conclusion (the surviving tokens keep their original position IDs): the rotary-encoding
 * tables the layers after the compression need for the rows of the re-assembled sequence.
 * Rotary position embedding as published: pair i of a head's dimensions turns by
 * pos * base^(-2 i / head_dim).
 *   pos      device, [n_rows] int32 position IDs (tc_reassemble's `pos`, flattened over the batch)
 *   head_dim even, >= 2;  base > 1 (10000 for LLaVA-1.5's language model)
 *   cos_out, sin_out  device, [n_rows, head_dim / 2] float32 out
 * The angle is formed in double precision, so the tables are good to float32 rounding for any
 * position.  Allocates nothing, only enqueues.
 */
tc_status tc_rope_tables(const int32_t* pos, int64_t n_rows, int32_t head_dim, float base,
                         float* cos_out, float* sin_out, void* stream);

/*
 * Number of image groups tc_score / tc_carve run side by side (1..16, default 4; the paper has
 * no counterpart).  The batch is cut into that many contiguous groups whose chains (Gram ->
 * eigen-solve -> scores, and in tc_carve the selection and gather as well) are enqueued on
 * internal streams forked from `stream` and joined back into it, so that the
 * one-block-per-image solver kernels of one group overlap the products of another.  With four
 * or more groups and 32 or more images they start in waves (two; four from eight groups on), a
 * wave's Gram products behind the previous wave's, so that the groups are not all in the same
 * phase of the chain.
 * Results do not depend on the setting.  The setting is process-wide state (one value for all
 * threads and devices), and calls that use groups are serialised on a lock while they enqueue.
 * Each group costs the host a few dozen launches per call: more than four groups pay only when
 * the call is replayed from a CUDA graph, where sixteen is the measured optimum at B = 64
 * (1.29 ms per carve against 1.31 ms with eight and 1.35 ms with eight in one wave).
 */
tc_status tc_set_groups(int32_t groups);

/*
 * Test hook, not part of the method: while `on` is non-zero every launcher that needs a TMA
 * tensor map is refused on the host (as if the driver's encode entry point were missing), so
 * that the calls' error paths can be exercised without faulting a GPU: tc_score / tc_carve /
 * tc_gram / tc_matmul_f32x3 / tc_probe then return TC_ERR_CUDA, leave no kernel of the refused
 * step enqueued, join their internal streams, and tc_score / tc_carve set img_status of the
 * images they did not reach.  Process-wide; returns TC_OK.
 */
tc_status tc_test_fail_tensor_maps(int32_t on);

/*
 * Optional event profile (diagnostics; the paper has no counterpart).  Between
 * tc_profile_begin() and tc_profile_end() every kernel launch of the library is bracketed by
 * CUDA events on its stream.  tc_profile_end() waits for those events and returns, per kernel
 * class (0 .. TC_N_KERNEL_CLASSES-1, named by tc_kernel_class_name), the summed device time in
 * milliseconds and the number of launches, in the HOST arrays ms[n], launches[n]
 * (n >= TC_N_KERNEL_CLASSES).  Not thread-safe against concurrent carve calls.
 */
#define TC_N_KERNEL_CLASSES 15
int32_t tc_profile_begin(void);
int32_t tc_profile_end(double* ms, int64_t* launches, int32_t n);
const char* tc_kernel_class_name(int32_t cls);

/* Number of kernels the library has launched in this process so far (diagnostics). */
int64_t tc_launch_count(void);

const char* tc_status_string(int32_t status);
int32_t tc_version(void);

#ifdef __cplusplus
}
#endif
#endif /* TOKENCARVE_H */
