/* critiprefill.h -- C ABI of the B200 (sm_100a) CritiPrefill prefill hot path.
 *
 * The library computes, for one attention layer,
 *   (1) segment-wise query criticality  ln S[j,b]   (paper Algorithm 1),
 *   (2) the per-segment critical block list          (Algorithm 2, line 8),
 *   (3) causal GQA attention over the listed blocks  (Algorithm 2, lines 6-13),
 * and, as the baseline the method is compared with, dense causal attention (Eq. 2).
 *
 * General conventions
 *   - Every pointer argument except `p`, `bytes_out` and `status_out` is a DEVICE pointer
 *     owned by the caller.  The library allocates no device memory, frees nothing and keeps
 *     no state between calls (one exception: critiprefill_estimate_static remembers, per device,
 *     the address of its built-in scratch array; see there).
 *   - Calls validate their arguments on the host, enqueue kernels on `cuda_stream`
 *     (a cudaStream_t passed as void*; NULL = the default stream) and return without
 *     synchronising.  Outputs are valid once the stream reaches that point.
 *     The calls (critiprefill_device_status excepted) only enqueue kernels and one small memset, so a stream
 *     that is being captured into a CUDA graph may carry them; the graph then refers to the buffers given at
 *     capture time (tensor maps are encoded on the host from those pointers).
 *   - Return value: a cp_status.  Conditions only the device can see (a block list that
 *     breaks its contract, a pipeline wait that ran out) are recorded in the first word of
 *     the workspace; read it with critiprefill_device_status.  Kernels never trap or assert.
 *   - Tensor layout: Q and O are [batch, n_q_heads, seq_len, head_dim], K and V are
 *     [batch, n_kv_heads, seq_len, head_dim]; the three outer strides are given in ELEMENTS
 *     in cp_params, head_dim is contiguous.  Base pointers must be 16-byte aligned and the
 *     strides multiples of 8 elements (bf16, fp16) / 4 elements (fp32).
 *   - Notation: n1 = ceil(seq_len / segment_size), n2 = ceil(seq_len / block_size) (the paper writes
 *     exact divisions; a remainder leaves a shorter last segment / block),
 *     r = segment_size / block_size (blocks that overlap a segment), k = budget_blocks,
 *     g = n_q_heads / n_kv_heads; query head h uses KV head h / g.
 *   - Requirements (else CP_ERR_SHAPE): segment_size % block_size == 0,
 *     n_q_heads % n_kv_heads == 0, k >= r (a budget beyond the visible blocks selects them all).
 *   - Supported (else CP_ERR_UNSUPPORTED): head_dim 64 or 128; n2 <= 8192 for estimate and select;
 *     the tensor-core attention path needs bf16 or fp16, head_dim 128, segment_size % 128 == 0 and
 *     block_size in {32, 64, 128}; everything else runs on a plain SIMT kernel.
 */
#ifndef CRITIPREFILL_H_
#define CRITIPREFILL_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  CP_OK = 0,
  CP_ERR_NULL = 1,        /* a required pointer is NULL */
  CP_ERR_SHAPE = 2,       /* sizes violate the divisibility / range requirements */
  CP_ERR_UNSUPPORTED = 3, /* valid problem outside the implemented envelope */
  CP_ERR_WORKSPACE = 4,   /* ws is NULL, misaligned (256 B) or smaller than workspace_bytes */
  CP_ERR_CUDA = 5,        /* a CUDA runtime/driver call failed (launch, tensor-map encode) */
  CP_ERR_TIMEOUT = 6,     /* device: a bounded pipeline wait expired; outputs are invalid */
  CP_ERR_BOUNDS = 7,      /* device: a block list broke its contract; that segment was skipped */
  CP_ERR_STATIC_LIMIT = 8 /* critiprefill_estimate_static: problem needs more scratch than the built-in array holds */
} cp_status;

typedef enum { CP_BF16 = 0, CP_F32 = 1, CP_F16 = 2 } cp_dtype;   /* fp16 is the paper's own precision (Section 3.1.3) */

enum {
  CP_FLAG_MASK_BEFORE_SOFTMAX = 1, /* estimate: normalise each score map over visible blocks only */
  CP_FLAG_FORCE_SIMT = 2,          /* attention: use the SIMT kernel even where tensor cores apply */
  CP_FLAG_TEST_WITHHOLD_V = 4,     /* test hook for the bounded waits of the tensor-core kernel: V tiles are
                                      never loaded, so a pipeline wait expires after about 2 s, the kernel
                                      drains and the status block reads CP_ERR_TIMEOUT (outputs invalid) */
  CP_FLAG_FORCE_SPLIT_SCORE = 16,  /* estimate: take the two-kernel score path (tensor-core log-sum-exps + exact logits of
                                      the visible blocks) whatever the size of the score map; without the flag it is used
                                      from a few million scores up, where it is faster (16-bit inputs, head_dim 128) */
  CP_FLAG_SUMMARIES_READY = 32,    /* estimate: the workspace already holds the representatives of these Q and K, written by
                                      critiprefill_project_qk with the same parameters: skip the pass over Q and K */
  CP_FLAG_SHARED_GROUP_LISTS = 8   /* select: one list per KV group instead of one per query head -- the g query
                                      heads of a KV head all receive the list selected from the element-wise
                                      maximum of their scores (a variant; the paper describes a single head) */
};

typedef struct {
  int32_t batch, n_q_heads, n_kv_heads, seq_len, head_dim;
  int32_t segment_size, block_size, budget_blocks; /* k = budget tokens / block_size */
  int32_t dtype;                                   /* cp_dtype of Q, K, V, O */
  int32_t flags;                                   /* CP_FLAG_* */
  int64_t q_stride[3], k_stride[3], v_stride[3], o_stride[3]; /* batch, head, token (elements) */
  float est_scale; /* multiplies the four estimation logits; 1.0 = Algorithm 1 as printed */
  float sm_scale;  /* attention logit scale, 1/sqrt(head_dim) in Eq. 2 / Algorithm 2 line 10 */
  float alpha;     /* layer-fusion weight of the current layer (Algorithm 1 line 14; 0.25 in
                      Section 3.1.3), in [0, 1] (else CP_ERR_SHAPE); ignored when S_prev is NULL */
  int32_t forced_blocks; /* select: n_sink | (n_local << 16), normally 0.  The first n_sink blocks of the sequence
                            and the n_local blocks right before each segment are always listed, like the diagonal
                            blocks, and count against k; requires n_sink + n_local <= k - r (else CP_ERR_SHAPE).
                            A variant: the paper fixes no sink or local blocks */
} cp_params;

/* Bytes of scratch (`ws`) the calls below need for these parameters; the same buffer serves
 * all of them.  `ws` must be 256-byte aligned.  Its first 256 bytes are the device status
 * block, which the caller zeroes once (cudaMemset) before the first call; the attention calls
 * also keep their work-unit counter there and reset it themselves at every launch.  Calls that
 * may execute concurrently (different streams without ordering) need separate workspaces;
 * calls ordered on one stream can share one.  Host pointers. */
int critiprefill_workspace_bytes(const cp_params* p, size_t* bytes_out);

/* Algorithm 1 (estimation of query criticality in one layer).
 *   Q, K    in   device, layout above.  V is not read by Algorithm 1.
 *   S_prev  in   device, nullable: ln S returned for the previous layer, [B,Hq,n1,n2] fp64.
 *                NULL = first layer / no fusion (alpha treated as 1).
 *   S_out   out  device, [B,Hq,n1,n2] fp64: NATURAL LOG of the criticality score,
 *                ln( alpha*S + (1-alpha)*S' ); blocks that start at or after the end of the
 *                segment (causal mask, line 13) hold -inf.  May not alias S_prev.
 * Steps: per-channel max/min of each query segment and key block (lines 3-8) into ws, four
 * dot-product logit maps scaled by est_scale and their row softmaxes over all n2 blocks
 * (lines 9-10), (S1+S3)/2, (S2+S4)/2 and their maximum (lines 11-12), mask (13), fusion (14).
 * Arithmetic: fp64 on the representatives (which are exact in the input dtype). */
int critiprefill_estimate(const cp_params* p, const void* Q, const void* K, const double* S_prev,
                          double* S_out, void* ws, size_t ws_bytes, void* cuda_stream);

/* critiprefill_estimate for callers that cannot allocate device memory.  (The paper has no
 * counterpart: this is a deployment convenience of this library, not part of the method.)
 * Meant for code that cannot obtain a workspace where it calls us -- a server whose memory
 * pool took the whole device at start-up, a loop that must not incur cudaMalloc's device-wide
 * synchronisation, a plug-in bound by its host's allocation rules.  Same arguments, results
 * and arithmetic as critiprefill_estimate, minus `ws`: the summaries go to an 8 MiB array
 * that is part of the library's device image (critiprefill_static_scratch_bytes(); every GPU
 * that loads the library holds it until the process exits).  8 MiB holds, for instance, 128K
 * tokens of 32 query / 8 KV heads at segment 1024 / block 128, but not at segment 512 / block 32.
 *   - The resolved address is cached per device for the life of the process; do not call this
 *     entry point again on a device after a cudaDeviceReset of that device.
 *   - Problems whose critiprefill_workspace_bytes exceeds that size return
 *     CP_ERR_STATIC_LIMIT and launch nothing.
 *   - The call allocates and frees nothing (no cudaMalloc/cudaFree, no allocating library
 *     routine).  The first call on each device resolves the array's device address with
 *     cudaGetSymbolAddress (that device must be current); make that first call during
 *     set-up, before any stream capture.
 *   - All calls on a device share the one array and it keeps the previous call's contents;
 *     the library clears the part that must start at zero.  Two calls whose kernels overlap
 *     on the GPU (different streams, no ordering between them) race on it: serialise them. */
int critiprefill_estimate_static(const cp_params* p, const void* Q, const void* K, const double* S_prev,
                                 double* S_out, void* cuda_stream);

/* Size in bytes of the built-in scratch array used by critiprefill_estimate_static. */
size_t critiprefill_static_scratch_bytes(void);

/* Algorithm 2, line 8: I_j = argtop_k(S[j], k) with the diagonal blocks always kept.
 *   S    in   device, [B,Hq,n1,n2] fp64 (as written by critiprefill_estimate)
 *   idx  out  device, [B,Hq,n1,k] int32: ascending block indices; the r_j blocks overlapping
 *             segment j ([j*r, min(n2,(j+1)*r)); r_j = r except in a short last segment) are
 *             always present and count against k; the other k-r_j entries are the
 *             strictly-past blocks with the largest S[j,b], ties to the larger b; entries
 *             beyond cnt are -1.  With CP_FLAG_SHARED_GROUP_LISTS the score of a block is the
 *             largest over the g query heads of the KV group and those heads share the list;
 *             forced_blocks adds always-kept sink / local blocks (see cp_params)
 *   cnt  out  device, [B,Hq,n1] int32 = min(k, number of blocks visible to segment j)
 * Exact (comparisons only). */
int critiprefill_select(const cp_params* p, const double* S, int32_t* idx, int32_t* cnt, void* ws,
                        size_t ws_bytes, void* cuda_stream);

/* Eq. 1 for queries and keys, fused with what Algorithm 1 needs from them: Q = W_Q X and K = W_K X on the tensor cores
 * (16-bit operands, fp32 accumulation), rotary position embedding in fp32 (rotate-half pairing: channel i with channel
 * i + head_dim/2, angle given by the caller's tables; the paper does not mention it, the models it evaluates apply it
 * here), results rounded once to the 16-bit dtype and stored -- and, from those stored values, the per-channel max / min
 * of every query segment and key block (Algorithm 1, lines 3-8) written to `ws`, so that a following
 * critiprefill_estimate with CP_FLAG_SUMMARIES_READY and the same `p` and `ws` need not read Q and K again.
 *   X          in   device, [batch, seq_len, d_model] contiguous, dtype as in p (bf16 or fp16)
 *   Wq, Wk     in   device, [n_q_heads*head_dim, d_model] and [n_kv_heads*head_dim, d_model], row-major
 *   rope_cos, rope_sin  in  device, nullable together: [seq_len, head_dim/2] fp32; NULL = no rotation (Eq. 1 as printed)
 *   Q_out, K_out  out  device, layouts given by p->q_stride / p->k_stride
 * Supported: head_dim 128, segment_size % 128 == 0, block_size in {32, 64, 128}, d_model % 64 == 0, seq_len >= 128
 * (else CP_ERR_UNSUPPORTED).  The representatives are bit-identical to what critiprefill_estimate computes from the
 * stored Q_out, K_out. */
int critiprefill_project_qk(const cp_params* p, const void* X, const void* Wq, const void* Wk, const float* rope_cos,
                            const float* rope_sin, int32_t d_model, void* Q_out, void* K_out, void* ws, size_t ws_bytes,
                            void* cuda_stream);

/* critiprefill_project_qk with the value projection of Eq. 1 in the same launch: V = W_V X, no rotation, rounded once and
 * stored with p->v_stride; Algorithm 1 takes nothing from V, so no representatives are formed for it.
 *   Wv     in   device, [n_kv_heads*head_dim, d_model] row-major;  V_out  out  device.  Both NULL = critiprefill_project_qk. */
int critiprefill_project_qkv(const cp_params* p, const void* X, const void* Wq, const void* Wk, const void* Wv,
                             const float* rope_cos, const float* rope_sin, int32_t d_model, void* Q_out, void* K_out,
                             void* V_out, void* ws, size_t ws_bytes, void* cuda_stream);

/* Query criticality of the LAST token, the decoding-phase use that Section 2.1 describes (the query of the last
 * token against the cached keys).  The paper gives no formula for it; this is Algorithm 1 on a segment that holds
 * that one token: Qmax = Qmin = q, every block is visible, no layer fusion.
 *   q_last  in   device, [batch, n_q_heads, head_dim] contiguous, dtype as in p
 *   K       in   device, layout and strides as in p (seq_len tokens)
 *   S_out   out  device, [B,Hq,n2] fp64: ln max( softmax_b(q.Kmax_b), softmax_b(q.Kmin_b) )
 * `ws` as for critiprefill_estimate (critiprefill_workspace_bytes of the same p is enough). */
int critiprefill_decode_estimate(const cp_params* p, const void* q_last, const void* K, double* S_out, void* ws,
                                 size_t ws_bytes, void* cuda_stream);

/* Critical blocks of the last token from critiprefill_decode_estimate's scores:
 *   idx  out  device, [B,Hq,k] int32 ascending, -1 padded: the last block (which holds the token) always, then the
 *             k-1 other blocks with the largest score, ties to the larger index (forced_blocks and
 *             CP_FLAG_SHARED_GROUP_LISTS apply as in critiprefill_select)
 *   cnt  out  device, [B,Hq] int32 = min(k, n2) */
int critiprefill_decode_select(const cp_params* p, const double* S, int32_t* idx, int32_t* cnt, void* ws,
                               size_t ws_bytes, void* cuda_stream);

/* Algorithm 2, lines 6-13, with token-level causality inside the listed blocks:
 *   O[t] = sum_{u in U_t} softmax_u(sm_scale * q_t.k_u) v_u,
 *   U_t  = { u <= t : floor(u/block_size) in idx[b,h,j,0:cnt] },  j = floor(t/segment_size).
 *   Q, K, V   in   device
 *   idx, cnt  in   device.  Contract per list (Algorithm 2 takes any index set I): 0 <= cnt <= k
 *                  entries, ascending, unique, each a block segment j can see, 0 <= b < min(n2, (j+1)*r).
 *                  Lists of the form critiprefill_select emits (past blocks, then exactly the diagonal
 *                  blocks) take the fast tile sequence; any other valid list is served element by
 *                  element masking (a listed diagonal block gets the causal mask wherever it sits).
 *                  A row that sees no key at all (possible only when diagonal blocks are left out)
 *                  gets O = 0 and lse = -inf.  A list that breaks the contract sets CP_ERR_BOUNDS in
 *                  the status block and its segment's rows of O are not written.
 *   O         out  device, same dtype and layout family as Q (o_stride)
 *   lse       out  device, nullable, [B,Hq,n] fp32: ln sum_{u in U_t} exp(sm_scale*q_t.k_u)
 * bf16 / fp16: operands in that type, fp32 accumulation, probabilities rounded to that type
 * before the PV product, O rounded to it.  fp32: plain fp32 arithmetic. */
int critiprefill_attention(const cp_params* p, const void* Q, const void* K, const void* V,
                           const int32_t* idx, const int32_t* cnt, void* O, float* lse, void* ws,
                           size_t ws_bytes, void* cuda_stream);

/* Eq. 2 with the causal mask (U_t = { u <= t }): the dense baseline, built on the same
 * pipeline as critiprefill_attention.  Arguments as above; segment_size / block_size /
 * budget_blocks are ignored apart from the shape requirements. */
int critiprefill_dense_attention(const cp_params* p, const void* Q, const void* K, const void* V,
                                 void* O, float* lse, void* ws, size_t ws_bytes,
                                 void* cuda_stream);

/* A packed batch of sequences of different lengths: one layer of the hot path (Algorithm 1, Algorithm 2 line 8,
 * Algorithm 2 lines 6-13) for each sequence.  The paper describes a single sequence; here every sequence is a problem
 * of its own: its segments and blocks are counted from its first token, its block indices are relative to that token,
 * and no query sees a key of another sequence.
 *   p           batch must be 1; seq_len = the LONGEST sequence (it sizes `ws`); the strides' batch entry is ignored,
 *               their head and token entries describe the packed tensors [total_tokens, heads, head_dim]
 *   cu_seqlens  in  HOST, n_seqs + 1 entries: 0, len_0, len_0 + len_1, ...; strictly increasing; len_i <= p->seq_len.
 *               Sequence i holds packed tokens [cu_seqlens[i], cu_seqlens[i+1])
 *   Q, K, V     in  device, packed;  O out device, packed;  lse out device, nullable, [Hq] x packed token:
 *               sequence i's part is the [Hq, len_i] array that starts at element Hq * cu_seqlens[i]
 *   S_prev      in  device, nullable; S_out, idx, cnt  out device: the per-sequence arrays of critiprefill_estimate /
 *               critiprefill_select ([Hq,n1_i,n2_i] fp64, [Hq,n1_i,k] int32, [Hq,n1_i] int32 with n1_i, n2_i from
 *               len_i) stored one after another in sequence order; critiprefill_varlen_sizes gives the totals
 * The sequences run one after another on `cuda_stream` through the same kernels as the single-sequence calls, so each
 * sequence's results are those of critiprefill_estimate + _select + _attention on its slice, bit for bit.
 * Errors: CP_ERR_SHAPE for a bad cu_seqlens or batch != 1; otherwise as the single-sequence calls. */
int critiprefill_prefill_varlen(const cp_params* p, const int32_t* cu_seqlens, int32_t n_seqs, const void* Q,
                                const void* K, const void* V, const double* S_prev, double* S_out, int32_t* idx,
                                int32_t* cnt, void* O, float* lse, void* ws, size_t ws_bytes, void* cuda_stream);

/* Element counts of the packed S (fp64), idx and cnt (int32) arrays of critiprefill_prefill_varlen.  Host pointers. */
int critiprefill_varlen_sizes(const cp_params* p, const int32_t* cu_seqlens, int32_t n_seqs, int64_t* s_elems,
                              int64_t* idx_elems, int64_t* cnt_elems);

/* Synchronises `cuda_stream`, copies the device status word (a cp_status: CP_OK, CP_ERR_TIMEOUT
 * or CP_ERR_BOUNDS; sticky until the caller zeroes the status block) to *status_out (host). */
int critiprefill_device_status(const void* ws, int32_t* status_out, void* cuda_stream);

/* Static, NUL-terminated description of a cp_status value. */
const char* critiprefill_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* CRITIPREFILL_H_ */
