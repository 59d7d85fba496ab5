/*
 * pafu.h - C ABI of the PaFu-KV inference hot path on NVIDIA B200 (sm_100a).
 *
 * The path is the per-layer cache update and attention of the paper's inference
 * procedure (Algorithm 2; Sec. 3.3, 3.4):
 *
 *     score   -> salience of every cached token from the S-MLP head
 *     select  -> indices of the retained tokens (sink + top-k salient + recent)
 *     compact -> KV <- Select(KV; ids), SL <- Select(SL; ids)
 *     attend  -> the new chunk's queries over [retained cache ; chunk's own tokens]
 *
 * Conventions that hold for every entry point
 *   - Plain C; every function returns a pafu_status and never throws or aborts.
 *   - No function allocates or frees device memory and none synchronises the device,
 *     unless its comment says otherwise.  All GPU work is enqueued on the caller's CUDA
 *     stream, passed as `void*` (a cudaStream_t; NULL is the default stream).
 *   - The caller owns every buffer.  "device" pointers are CUDA device pointers valid
 *     on the current device; "host" pointers are ordinary host memory read before the
 *     call returns.  Device buffers must be 16-byte aligned.
 *   - bf16 tensors are raw 16-bit patterns (`uint16_t`).  Token tensors are token-major
 *     `[tokens, n_heads, d_head]`, contiguous (d_model = n_heads * d_head elements per
 *     row) - the merged layout the paper feeds to the S-MLP (Appendix A, "S-MLP").
 *   - Several independent streams (a ragged batch) are packed back to back: stream s owns
 *     token rows [cu[s], cu[s+1]) of a tensor, `cu` being a host prefix array of
 *     n_streams + 1 entries starting at 0.  At most PAFU_MAX_STREAMS streams.
 *   - Argument errors are found on the host before anything is launched; in that case no
 *     output is touched.
 *   - Kernels that wait on asynchronous copies bound every wait.  A wait that runs out
 *     records a code in the workspace header and the kernel returns; see
 *     pafu_workspace_status().
 */
#ifndef PAFU_H_
#define PAFU_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define PAFU_MAX_STREAMS 32
#define PAFU_MAX_LAYERS 64

typedef int32_t pafu_status;
enum {
    PAFU_OK = 0,
    PAFU_ERR_INVALID_ARG = 1,        /* null pointer, negative size, bad enum, bad prefix array */
    PAFU_ERR_BAD_BUDGET = 2,         /* negative budget / sink / recent */
    PAFU_ERR_UNSUPPORTED_SHAPE = 3,  /* a dimension outside the supported set (see each call) */
    PAFU_ERR_WORKSPACE_TOO_SMALL = 4,
    PAFU_ERR_MISALIGNED = 5,         /* a device pointer is not 16-byte aligned */
    PAFU_ERR_CUDA = 6,               /* a CUDA runtime/driver call failed (launch error, no device) */
    PAFU_ERR_TIMEOUT = 7,            /* a bounded device-side wait ran out (pafu_workspace_status) */
    PAFU_ERR_TOO_LARGE = 8           /* exceeds pafu_chunk_attn_noalloc's built-in scratch, or a pafu_cache's capacity */
};

/* Activation between the two linear layers of the salience head. */
enum { PAFU_ACT_GELU = 0 /* x * Phi(x), exact erf form */, PAFU_ACT_SILU = 1 /* paper's S-MLP */ };
/* Map applied to the mean of the head's outputs. */
enum { PAFU_FINAL_NONE = 0, PAFU_FINAL_SIGMOID = 1 };

/* Geometry of one call.  cu_T: cache tokens per stream before pruning; cu_Lq: chunk (query)
 * tokens per stream.  Both are HOST arrays of n_streams + 1 non-decreasing prefix offsets.
 * A function that does not need one of them ignores it (may be NULL). */
typedef struct pafu_shape {
    int32_t n_heads;
    int32_t d_head;
    int32_t n_streams;
    const int64_t* cu_T;   /* host */
    const int64_t* cu_Lq;  /* host */
} pafu_shape;

/* Salience Estimation Head (Sec. 3.3; Appendix A "S-MLP"): two linear layers with an
 * activation in between; the d_out outputs are averaged into one scalar per token.
 * Weights use the torch.nn.Linear layout.  All four pointers are DEVICE bf16 arrays;
 * b1 and b2 may be NULL (no bias).  The paper's head is d_in = 4608, d_hidden = 1024,
 * d_out = 12, SiLU, no final map. */
typedef struct pafu_head {
    int32_t d_in;
    int32_t d_hidden;
    int32_t d_out;
    int32_t act;           /* PAFU_ACT_* */
    int32_t final;         /* PAFU_FINAL_* */
    const uint16_t* w1;    /* device [d_hidden, d_in] */
    const uint16_t* b1;    /* device [d_hidden] or NULL */
    const uint16_t* w2;    /* device [d_out, d_hidden] */
    const uint16_t* b2;    /* device [d_out] or NULL */
} pafu_head;

/* Retention rule of one stream, in absolute token counts. */
typedef struct pafu_policy {
    int64_t n_sink;    /* leading tokens always kept (frame sink, Sec. 4.1) */
    int64_t n_recent;  /* trailing tokens always kept (the newest chunk survives one round, Alg. 2) */
    int64_t budget;    /* tokens kept in total; T <= budget keeps all T */
} pafu_policy;

/* Library version (major * 1000 + minor). */
int32_t pafu_version(void);

/* Static, human-readable name of a status code. */
const char* pafu_status_string(pafu_status s);

/* Number of tokens each stream keeps, as a prefix array.
 * cu_B (HOST, out, n_streams + 1 entries): cu_B[0] = 0, cu_B[s+1] - cu_B[s] = min(budget_s, T_s).
 * `policy` is a HOST array of n_streams entries.  Pure host arithmetic. */
pafu_status pafu_kept_counts(const pafu_shape* shape, const pafu_policy* policy, int64_t* cu_B);

/* Bytes of device scratch that pafu_score / pafu_select / pafu_chunk_attn / pafu_step need
 * for this geometry (`head` and `policy` may be NULL when the corresponding step is not
 * used).  Returns 0 on invalid arguments.  The workspace must be 256-byte aligned; its
 * first 256 bytes are a status header which the caller zeroes once after allocating.  The
 * library keeps a time-out code, diagnostic counters and the work counters of pafu_step's row
 * gather there (the latter return to zero at the end of every call); one workspace serves one
 * call at a time - calls that may overlap on the GPU need a workspace each. */
size_t pafu_workspace_bytes(const pafu_shape* shape, const pafu_policy* policy,
                            const pafu_head* head);

/* Reads the workspace's status header.  SYNCHRONISES `stream` (one 4-byte device-to-host
 * copy).  Returns PAFU_OK, or PAFU_ERR_TIMEOUT if a kernel gave up on a bounded wait since
 * the header was last zeroed (the outputs of that launch are then undefined). */
pafu_status pafu_workspace_status(const void* ws, void* stream);

/* Diagnostic counters of the workspace's status header, accumulated by pafu_chunk_attn (d_head
 * 128) since the header was last zeroed.  SYNCHRONISES `stream`.  The attention kernel keeps a
 * running row maximum per query (the max-subtracted softmax of Sec. 3.2 evaluated tile by tile)
 * and only re-bases it when it must; the counters say how often each path ran, counted per
 * (32-row group, 64-key tile):
 *   counts[0]  tiles that took the exact pass because they open a run or end a key segment raggedly
 *   counts[1]  tiles that took the exact pass because a row sum showed a logit far above the
 *              running maximum
 *   counts[2]  tiles at which the output accumulator and the row sums were rescaled
 * counts is a HOST array of 3 entries.  Tests use it to show that an input reaches those paths.
 *
 * The header also holds a test hook: while its 32-bit word 32 is non-zero the attention kernel's
 * loader issues no copies, every consumer's bounded wait runs out and the launch ends with
 * PAFU_ERR_TIMEOUT in the header (outputs undefined).  It exists so that the time-out path can
 * be exercised without faulting the device; zero the header to return to normal operation. */
pafu_status pafu_workspace_counters(const void* ws, int64_t* counts, void* stream);

/* Step 1 - salience scores (Sec. 3.3, 3.4; Appendix A "S-MLP").
 * For every token row x of X: h = act(W1 x + b1); y = W2 h + b2; s = mean_o y_o;
 * s <- sigmoid(s) if head->final == PAFU_FINAL_SIGMOID.  bf16 operands, fp32 accumulation,
 * fp32 activation and output.
 *   head      HOST struct with DEVICE weight pointers
 *   X         device bf16 [n_tokens, ldx], row stride ldx >= d_in elements, ldx % 8 == 0
 *   scores    device fp32 [n_tokens], out
 *   ws        device workspace (pafu_workspace_bytes), ws_bytes its size
 * Supported: d_in % 64 == 0, d_hidden % 16 == 0 and <= 1024, d_out >= 1.
 * n_tokens == 0 is a no-op. */
pafu_status pafu_score(const pafu_head* head, const uint16_t* X, int64_t n_tokens, int64_t ldx,
                       float* scores, void* ws, size_t ws_bytes, void* stream);

/* Step 1 on the input the paper feeds its head (Sec. 3.3 "Salience Estimation Head"; Appendix A
 * "S-MLP": 4608 = 3 x 1536 inputs, 1024 hidden, 12 outputs, SiLU, mean over the outputs): token
 * t's feature vector is the concatenation [q_t, k_t, v_t] of its query, key and value rows.
 * The three matrices are read in place (no concatenated copy is made); everything else is as
 * pafu_score with x_t = [q_t, k_t, v_t], so W1's columns are ordered query, key, value.
 *   Q, K, V   device bf16 [n_tokens, ld] each, head->d_in / 3 features per row, ld % 8 == 0
 * Supported: head->d_in % 192 == 0 (each third a multiple of 64), else as pafu_score. */
pafu_status pafu_score_qkv(const pafu_head* head, const uint16_t* Q, const uint16_t* K, const uint16_t* V,
                           int64_t n_tokens, int64_t ld, float* scores, void* ws, size_t ws_bytes, void* stream);

/* Step 2 - retained indices (Sec. 3.4 inference paragraph; Algorithm 2 "Top-k"; frame sink
 * Sec. 4.1).  Per stream with T tokens and (n_sink, n_recent, budget):
 *   T <= budget            : keep all T tokens;
 *   else n_recent' = min(n_recent, budget), n_sink' = min(n_sink, budget - n_recent'),
 *        k = budget - n_sink' - n_recent', and the kept set is
 *        [0, n_sink') U top-k of scores[n_sink' : T - n_recent') U [T - n_recent', T).
 * Ranking is by fp32 value, higher first; equal values (-0 == +0) go to the lower index;
 * NaN ranks below every number.  The result is exact and deterministic.
 *   scores    device fp32 [cu_T[n_streams]], packed over streams
 *   policy    HOST array [n_streams]
 *   idx       device int32 [cu_B[n_streams]], out: per stream, stream-local token indices
 *             in strictly ascending order at offset cu_B[s] (cu_B from pafu_kept_counts)
 * Each stream needs T < 2^31. */
pafu_status pafu_select(const float* scores, const pafu_shape* shape, const pafu_policy* policy,
                        int32_t* idx, void* ws, size_t ws_bytes, void* stream);

/* Step 3 - KV <- Select(KV; ids), SL <- Select(SL; ids) (Algorithm 2).
 * For stream s and i in [0, B_s): Kc[cu_B[s] + i, :] = K[cu_T[s] + idx[cu_B[s] + i], :], same
 * for V and, when SL and SLc are both non-NULL, for the fp32 salience list.  Raw copies,
 * bit exact.  Out of place: outputs must not overlap inputs.
 *   K, V      device bf16 [cu_T[n_streams], n_heads, d_head]
 *   idx       device int32 as written by pafu_select (values must lie in [0, T_s))
 *   Kc, Vc    device bf16 [cu_B[n_streams], n_heads, d_head], out
 * Supported: n_heads * d_head % 8 == 0. */
pafu_status pafu_compact(const uint16_t* K, const uint16_t* V, const float* SL, const int32_t* idx,
                         const pafu_shape* shape, const pafu_policy* policy,
                         uint16_t* Kc, uint16_t* Vc, float* SLc, void* stream);

/* Step 3 for every layer at once.  The paper scores and selects at the final layer only and
 * reuses the indices for all layers (Sec. 3.3: the Top-k sets of the layers agree at t_0; Sec. 3.4:
 * the head sits in the final layer), so one index list prunes n_layers caches.  Exactly
 * pafu_compact applied to each (K[l], V[l]) -> (Kc[l], Vc[l]) with the same idx, in one launch;
 * SL -> SLc (both or neither NULL) is compacted once.
 *   K, V, Kc, Vc   HOST arrays of n_layers DEVICE pointers (read before the call returns), each
 *                  tensor laid out as for pafu_compact; n_layers <= PAFU_MAX_LAYERS */
pafu_status pafu_compact_layers(const uint16_t* const* K, const uint16_t* const* V, int32_t n_layers,
                                const float* SL, const int32_t* idx, const pafu_shape* shape,
                                const pafu_policy* policy, uint16_t* const* Kc, uint16_t* const* Vc,
                                float* SLc, void* stream);

/* Step 4 - chunk attention over the retained cache (Sec. 3.2 for the operator
 * P = softmax(Q K^T / sqrt(D)); Eq. 2 / Eq. 7 for what it ranges over).
 * Per stream s, head n, query row i: o_i = sum_j softmax_j(scale * q_i . k_j) v_j where j runs
 * over the B_s retained tokens (Kc, Vc) and then the stream's own Lq_s chunk tokens (Kq, Vq).
 * No mask: the chunk is bidirectional and sees the whole retained cache.  bf16 operands,
 * fp32 accumulation and softmax; probabilities are rounded to bf16 before the P V product.
 *   Q         device bf16 [cu_Lq[n_streams], n_heads, d_head]
 *   Kc, Vc    device bf16 [cu_B[n_streams], n_heads, d_head]
 *   cu_B      HOST prefix array [n_streams + 1] of retained tokens
 *   Kq, Vq    device bf16 [cu_Lq[n_streams], n_heads, d_head]; both NULL = no chunk segment
 *   scale     softmax scale; 0 means 1 / sqrt(d_head)
 *   O         device bf16 [cu_Lq[n_streams], n_heads, d_head], out
 *   LSE       device fp32 [n_heads, cu_Lq[n_streams]] log-sum-exp of the scaled logits, or NULL
 * A query with no keys at all gets o = 0 and LSE = -inf.  Supported: d_head in {64, 128}. */
pafu_status pafu_chunk_attn(const uint16_t* Q, const uint16_t* Kc, const uint16_t* Vc,
                            const int64_t* cu_B, const uint16_t* Kq, const uint16_t* Vq,
                            const pafu_shape* shape, float scale, uint16_t* O, float* LSE,
                            void* ws, size_t ws_bytes, void* stream);

/* Step 4 without step 3 - chunk attention that reads the retained tokens through the index list
 * ("index-based cache management": Sec. 3.4, Eq. 7 restricts attention to the index set I_s of the
 * full cache instead of to a copied cache).  Computes exactly what pafu_compact followed by
 * pafu_chunk_attn computes - the outputs are bit-identical - but K and V are the UNCOMPACTED
 * cache and the loader fetches rows idx[.] of it, so no compacted copy is written or read (the
 * attention itself runs about a tenth slower than on a compacted cache).
 *   K, V      device bf16 [cu_T[n_streams], n_heads, d_head], the cache before pruning
 *   idx       device int32 [cu_B[n_streams]] as written by pafu_select: per stream, stream-local
 *             token indices in [0, T_s), at offset cu_B[s]
 *   cu_B      HOST prefix array of retained tokens (pafu_kept_counts); B_s <= T_s
 *   shape     needs both cu_T and cu_Lq
 * Everything else as pafu_chunk_attn.  Supported: d_head = 128; every stream with queries needs
 * at least one key; K and V smaller than 64 GiB each. */
pafu_status pafu_chunk_attn_indexed(const uint16_t* Q, const uint16_t* K, const uint16_t* V, const int32_t* idx,
                                    const int64_t* cu_B, const uint16_t* Kq, const uint16_t* Vq,
                                    const pafu_shape* shape, float scale, uint16_t* O, float* LSE,
                                    void* ws, size_t ws_bytes, void* stream);

/* Chunk attention without a workspace - the paper has no counterpart; this entry point exists
 * for callers that are not allowed to allocate device memory: code running inside another
 * framework's memory plan or a fixed-memory service, plug-ins handed only their input and
 * output buffers, and anything else that must not call cudaMalloc (directly or through an
 * allocating library) on its hot path.  It computes exactly what pafu_chunk_attn computes
 * (same arguments, same layouts, d_head = 128 only, every stream needs at least one key), but
 * the scratch the kernel needs lives in a device array built into the library:
 * PAFU_NOALLOC_SCRATCH_BYTES bytes that every GPU which loads the library holds until the
 * process exits.  The call allocates and frees nothing.
 *   - Limit: sum over streams of query rows, times n_heads, must not exceed
 *     PAFU_NOALLOC_MAX_QUERY_HEAD_ROWS; larger problems return PAFU_ERR_TOO_LARGE and nothing
 *     is launched.  The built-in scratch holds the partial results of 31 thread blocks, so the
 *     kernel runs on at most 31 SMs: expect it to be several times slower than pafu_chunk_attn.
 *   - The first call on each device looks up the device address of the built-in array (a
 *     runtime query, no allocation).  Make that first call outside any stream capture.
 *   - All calls share the one array and it keeps whatever the last call left there; the call
 *     clears the part that must start at zero itself.  Two calls that overlap on the GPU (on
 *     different streams, or from different host threads) race on it: serialise them.
 *   - A bounded wait that runs out cannot be reported (there is no workspace to read back);
 *     use pafu_chunk_attn where that matters. */
#define PAFU_NOALLOC_SCRATCH_BYTES (8u * 1024u * 1024u)
#define PAFU_NOALLOC_MAX_QUERY_HEAD_ROWS 65536
pafu_status pafu_chunk_attn_noalloc(const uint16_t* Q, const uint16_t* Kc, const uint16_t* Vc,
                                    const int64_t* cu_B, const uint16_t* Kq, const uint16_t* Vq,
                                    const pafu_shape* shape, float scale, uint16_t* O, float* LSE,
                                    void* stream);

/* Arguments of one whole layer step (Algorithm 2's order: score, Top-k, Select, attend). */
typedef struct pafu_step_args {
    pafu_shape shape;
    const pafu_head* head;        /* host struct, device weights; d_in must equal n_heads*d_head */
    const pafu_policy* policy;    /* host [n_streams] */
    const uint16_t* K;            /* device [cu_T[n], N, D]: cache keys, also the head's input */
    const uint16_t* V;            /* device [cu_T[n], N, D] */
    const uint16_t* Q;            /* device [cu_Lq[n], N, D] */
    const uint16_t* Kq;           /* device [cu_Lq[n], N, D] */
    const uint16_t* Vq;           /* device [cu_Lq[n], N, D] */
    float scale;                  /* 0 = 1/sqrt(D) */
    float* scores;                /* device fp32 [cu_T[n]], out (also the salience list SL) */
    int32_t* idx;                 /* device int32 [cu_B[n]], out */
    uint16_t* Kc;                 /* device [cu_B[n], N, D], out */
    uint16_t* Vc;                 /* device [cu_B[n], N, D], out */
    float* SLc;                   /* device fp32 [cu_B[n]], out, or NULL */
    uint16_t* O;                  /* device [cu_Lq[n], N, D], out */
    float* LSE;                   /* device fp32 [N, cu_Lq[n]], out, or NULL */
    void* ws;                     /* device workspace */
    size_t ws_bytes;
} pafu_step_args;

/* Step 5 - the four steps in order on one stream.  Produces exactly what pafu_score,
 * pafu_select, pafu_compact and pafu_chunk_attn produce when called in sequence with the
 * same buffers (the salience head reads each token's K across all heads). */
pafu_status pafu_step(const pafu_step_args* args, void* stream);

/* The layer step without the compaction copy: score, Top-k, then pafu_chunk_attn_indexed on the
 * uncompacted cache (Algorithm 2 with Select(KV; ids) applied inside the attention's loader).
 * args->Kc, Vc, SLc are ignored (may be NULL); scores, idx, O (and LSE) are written and equal
 * pafu_step's bit for bit.  d_head = 128 only. */
pafu_status pafu_step_indexed(const pafu_step_args* args, void* stream);

/* pafu_step with timestamps: identical launches, plus five caller-created CUDA events
 * (HOST array of 5 cudaEvent_t passed as void*) recorded on `stream`: events 0 and 1 around the
 * score step, events 2 and 3 around selection + row gather (two launches that overlap: the
 * gather copies the always-kept rows while the selection runs, so no event can sit between
 * them; event 2 follows event 1 at once), event 4 after the attention.  Lets a caller attribute
 * the step's time to its kernels.  The events between the kernels do cost the overlap of each
 * kernel's set-up with its predecessor's end, so the parts sum to slightly more than pafu_step. */
pafu_status pafu_step_timed(const pafu_step_args* args, void* const* events, void* stream);

/* Bytes of device memory pafu_step_host needs as its arena for this geometry. */
size_t pafu_step_host_arena_bytes(const pafu_shape* shape, const pafu_policy* policy,
                                  const pafu_head* head);

/* pafu_step for callers whose tensors live in HOST memory.  Every tensor pointer in `args`
 * (K, V, Q, Kq, Vq, the head's weights; outputs scores, idx, O and, if non-NULL, Kc, Vc, SLc,
 * LSE) is a HOST pointer - pinned memory makes the copies asynchronous.  args->ws/ws_bytes
 * are ignored.  The call copies the inputs into `arena` (device, 256-byte aligned, at least
 * pafu_step_host_arena_bytes), runs pafu_step there, copies the outputs back and
 * SYNCHRONISES `stream` before returning, so the host outputs are valid on return.
 * Returns PAFU_ERR_TIMEOUT if a bounded device wait ran out. */
pafu_status pafu_step_host(const pafu_step_args* args, void* arena, size_t arena_bytes,
                           void* stream);

/* pafu_step_host without the final synchronisation, for callers that keep several steps in flight
 * (two streams with an arena each: the copies of one step then overlap the kernels of the other
 * and the host link, not the sum of link and kernels, sets the pace).  Everything is enqueued on
 * `stream` and the call returns; the host outputs, and *timeout_word, are valid once the caller
 * has synchronised `stream`.
 *   timeout_word   HOST int32 (pinned memory for a truly asynchronous copy), out: 0, or the code of
 *                  a bounded device wait that ran out (treat non-zero as PAFU_ERR_TIMEOUT)
 * The argument structs, the prefix arrays and the host buffers must stay valid until then, and the
 * arena must not be used by another call in the meantime. */
pafu_status pafu_step_host_async(const pafu_step_args* args, void* arena, size_t arena_bytes,
                                 void* stream, int32_t* timeout_word);

/* The rolling KV cache of Algorithm 2 for one stream and all layers, and its update once a chunk
 * has been generated (Sec. 3.3: the salience head sits in the final layer and its Top-k prunes
 * every layer's cache; Algorithm 2: "if |KV| = L: ids <- Top-k(SL); KV <- Select(KV; ids);
 * SL <- Select(SL; ids)", then KV.append(kv), SL.append(s)).
 * The cache lives in two sets of buffers; a pruning gathers from the current set into the other
 * and makes that one current (rows are never moved inside a buffer).  All counters are host-side. */
typedef struct pafu_cache {
    int32_t n_layers;        /* <= PAFU_MAX_LAYERS */
    int32_t n_heads, d_head; /* n_heads * d_head % 8 == 0 */
    int32_t cur;             /* in/out: which buffer set (0 or 1) holds the cache */
    int64_t capacity;        /* L: tokens a buffer holds */
    int64_t n_sink;          /* attention-sink prefix that every pruning keeps */
    int64_t T;               /* in/out: tokens in the cache, <= capacity */
    uint16_t* const* K[2];   /* HOST arrays of n_layers DEVICE pointers, each bf16 [capacity, n_heads, d_head] */
    uint16_t* const* V[2];
    float* SL[2];            /* device fp32 [capacity]: the salience list carried with the cache */
    int32_t* idx;            /* device int32 [capacity], 16-byte aligned: the index list of the last pruning */
} pafu_cache;

/* One chunk's update, enqueued on `stream` (nothing is synchronised; the host fields of `cache`
 * are updated before the call returns and describe the cache once the stream has caught up):
 *   1. if T + chunk > capacity: idx <- sink prefix + Top-k of SL[0:T] with k such that
 *      capacity - chunk tokens stay (ties to the lower index, ascending order: pafu_select with
 *      n_recent = 0); every layer's K and V and SL are gathered through idx into the other buffer
 *      set (pafu_compact_layers); cur flips; T <- capacity - chunk;
 *   2. the chunk's scores s = S-MLP([q, k, v]) (pafu_score_qkv on the final layer's rows) are
 *      written to SL[cur][T : T + chunk];
 *   3. every layer's new rows are copied to K[cur][l][T : T + chunk], V[cur][l][...]; T += chunk.
 *   head            as for pafu_score_qkv (d_in = 3 * n_heads * d_head)
 *   Qs, Ks, Vs      device bf16 [chunk, n_heads, d_head]: the final layer's rows the head reads
 *   Knew, Vnew      HOST arrays of n_layers DEVICE pointers, each bf16 [chunk, n_heads, d_head]
 *   pruned          host out, may be NULL: 1 if step 1 ran (cache->idx then holds capacity - chunk indices)
 *   ws, ws_bytes    as for pafu_score_qkv
 * Errors (before anything is enqueued): PAFU_ERR_TOO_LARGE if chunk > capacity,
 * PAFU_ERR_INVALID_ARG for NULL or inconsistent fields (cur not 0/1, T outside [0, capacity], the
 * two buffer sets sharing a pointer), PAFU_ERR_MISALIGNED, PAFU_ERR_UNSUPPORTED_SHAPE. */
pafu_status pafu_cache_update(pafu_cache* cache, const pafu_head* head,
                              const uint16_t* Qs, const uint16_t* Ks, const uint16_t* Vs,
                              const uint16_t* const* Knew, const uint16_t* const* Vnew, int64_t chunk,
                              int32_t* pruned, void* ws, size_t ws_bytes, void* stream);

/* Teacher-side salience target - Spatialtemporal-balanced Salience Estimation (Sec. 3.2, Eq. 4
 * and Eq. 5; Algorithm 3).  With P = softmax(scale * Q K^T) per head over the whole sequence of L
 * tokens (bidirectional) and blocks of block_len tokens, key j gets
 *   low_j  = mean over heads of max_i P[n,i,j] over the queries i of LATER blocks,
 *   diag_j = the same over the queries of j's OWN block,
 *   up_j   = the same over the queries of EARLIER blocks   (an empty set of queries gives 0),
 * and s_j = (diag + low) / 2 for j < block_len, (up + diag + low) / 3 for
 * block_len <= j < L - block_len, (diag + up) / 2 for the rest (the first matching case when
 * L < 2 * block_len).  P is never written: the kernel needs only each row's log-sum-exp.
 *   Q, K      device bf16 [L, n_heads, d_head]
 *   LSE       device fp32 [n_heads, L]: log-sum-exp of scale * q_i . k_j over all L keys, as
 *             pafu_chunk_attn writes it for the same Q, K and scale; NULL = computed here with the
 *             attention kernel (costs a full attention pass and scratch for its output)
 *   s         device fp32 [L], out
 *   comp      device fp32 [3, L], out: low, diag, up; or NULL
 *   gmax      device fp32 [L], out, or NULL: mean over heads of max_i P[n,i,j] over ALL queries -
 *             global max pooling, the "Max" alternative of the paper's ablation (Sec. 4.3, Table 3)
 *   gavg      device fp32 [L], out, or NULL: mean over heads and over ALL queries of P[n,i,j] -
 *             global average pooling, the "Avg" alternative of the same ablation; asking for it
 *             costs one exponential per (query, key, head) on top of the contraction
 *   ws        device workspace of pafu_sse_workspace_bytes(...), 256-byte aligned, status header
 *             (first 256 bytes) zeroed by the caller; read it back with pafu_workspace_status
 * Supported: d_head = 128, L < 2^31.  fp32 accumulation; results agree with the definition to
 * about 1e-5 relative (the logits' rounding), not bit for bit. */
size_t pafu_sse_workspace_bytes(int64_t L, int32_t n_heads, int32_t d_head, int64_t block_len);
pafu_status pafu_sse(const uint16_t* Q, const uint16_t* K, const float* LSE, int64_t L,
                     int32_t n_heads, int32_t d_head, int64_t block_len, float scale,
                     float* s, float* comp, float* gmax, float* gavg, void* ws, size_t ws_bytes, void* stream);

/* The salience target in Algorithm 3's order of operations.  Algorithm 3 averages the attention
 * weights over the heads BEFORE it takes the maximum over a block class's queries, while Eq. 4
 * takes each head's maximum first and then the mean (pafu_sse follows Eq. 4; for one head the two
 * are the same).  With a[i,j] = mean over heads of P[n,i,j]:
 *   low_j / diag_j / up_j = max of a[i,j] over the queries i of later / the same / earlier blocks
 * and s_j by Eq. 5 as in pafu_sse.  Every value is <= the corresponding value of pafu_sse.
 * Arguments as pafu_sse (without gmax and gavg); the workspace is the one of
 * pafu_sse_workspace_bytes.  Needs one exponential per (query, key, head) and runs on mma.sync
 * tiles: a comparison variant, several times slower than pafu_sse. */
pafu_status pafu_sse_mean_first(const uint16_t* Q, const uint16_t* K, const float* LSE, int64_t L,
                                int32_t n_heads, int32_t d_head, int64_t block_len, float scale,
                                float* s, float* comp, void* ws, size_t ws_bytes, void* stream);

#ifdef __cplusplus
}
#endif
#endif  /* PAFU_H_ */
