/*
 * stief.h -- C boundary of the B200 (sm_100a) library for decode attention over a KV cache that is
 * stored, per KV head, as projections onto column-orthonormal bases:
 *
 *     K_down = K U_k  in R^{n x r_k},   V_down = V U_v  in R^{n x r_v}          (paper Eq. 1, Sec. 3.2)
 *
 * and attended through the reconstructions K_tilde = K_down U_k^T, V_tilde = V_down U_v^T
 * (Eq. 2 / Eq. 7) with ordinary per-head attention softmax(q K_tilde^T / sqrt(d_h)) V_tilde (Eq. 18).
 * Because q K_tilde^T = (q U_k) K_down^T and p V_tilde = (p V_down) U_v^T, everything is evaluated
 * in the compressed space and the reconstructions are never formed.
 *
 * General rules
 *  - Every pointer below is a DEVICE pointer unless its name ends in _host.  The caller owns all
 *    memory.  No entry point allocates, frees or synchronises; all work is enqueued on `stream`
 *    (a cudaStream_t passed as void*; NULL = the legacy default stream).
 *  - bf16 tensors are passed as uint16_t* (raw bit patterns).  d_h must be 128.  Ranks must be one of
 *    32, 48, 64, 96, 128 (STIEF_ERR_UNSUPPORTED otherwise).  Ranks are per layer, equal across heads.
 *  - Return value: a stief_status for problems the host can see (bad arguments, launch failure).
 *    Problems only the device can see (a page id outside the pool, a position beyond the block
 *    table, a wait that ran out) are reported through the optional `status` word: a device int32
 *    the caller zeroes; the first error code wins; read it after synchronising.  A kernel that
 *    detects such a problem skips or redirects the offending access; it never traps.
 *  - Cache layout (bit-exact contract): pools are [num_pages][Hkv][64][r] bf16, r fastest.  Token t
 *    of sequence b, KV head h, lives at element ((block_table[b][t/64]*Hkv + h)*64 + t%64)*r.
 *    Rows of a page at or beyond the sequence length are unspecified and never influence a result.
 *  - Query head g reads KV head g / (Hq/Hkv) (contiguous GQA groups).
 *  - The softmax scale is always 1/sqrt(d_h) = 1/sqrt(128), never 1/sqrt(r_k): attention is defined
 *    on tensors of the original dimension (Eq. 7, Eq. 18).
 *  - RoPE (or any other positional map) is the caller's business: k, q arrive as the attention block
 *    sees them.
 */
#ifndef STIEF_H_
#define STIEF_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum stief_status {
  STIEF_OK = 0,
  STIEF_ERR_INVALID_ARG = 1,  /* NULL/misaligned pointer, bad shape                                    */
  STIEF_ERR_UNSUPPORTED = 2,  /* rank or head dimension not compiled in                                */
  STIEF_ERR_WORKSPACE = 3,    /* workspace too small for the requested number of splits                */
  STIEF_ERR_CUDA = 4,         /* a CUDA runtime/driver call failed (cudaGetLastError is left readable) */
  STIEF_ERR_BOUNDS = 5,       /* device-side: page id or position out of range (status word only)      */
  STIEF_ERR_TIMEOUT = 6,      /* device-side: a bounded wait on an async copy ran out (status word)    */
  STIEF_ERR_INFEASIBLE = 7    /* rank selection: no candidate pair fits the budget at some layer       */
};

#define STIEF_PAGE 64
#define STIEF_D_HEAD 128

/* One decoder layer's compressed cache and bases.
 * U_k: [Hkv][128][r_k] bf16 row-major (r fastest) with head stride uk_head_stride elements; stride 0
 * means one key basis shared by all heads of the layer (the paper's head-sharing scheme, Sec. 3.3).
 * U_v: [Hkv][128][r_v], per-head value bases (stride 128*r_v) or shared (stride 0).
 * A NULL basis means the library does not project that side: its rows arrive with r elements and are
 * stored and used as they are.  With r = 128 that is a layer that keeps keys or values full rank
 * (Algorithm 2); with r < 128 the projection has been folded into the model's linear layers (Sec. 3.3,
 * "Overheads": W_K U_k and W_Q U_k produce compressed keys and queries, W_V U_v compressed values, and
 * U_v^T W_O consumes the compressed attention output).  For a key side without basis q, k_new and K have
 * r_k elements per head; for a value side without basis v_new and V have r_v elements per head and the
 * outputs `out` are [B][Hq][r_v]: no back-projection is applied.
 * The same U buffers serve compression, query projection and back-projection.
 * Alignment: pools and bases 128 bytes. */
typedef struct stief_layer {
  int32_t Hq, Hkv, d;
  int32_t r_k, r_v;
  int32_t num_pages;
  const uint16_t* U_k;
  int64_t uk_head_stride;
  const uint16_t* U_v;
  int64_t uv_head_stride;
  uint16_t* k_pool; /* [num_pages][Hkv][64][r_k] */
  uint16_t* v_pool; /* [num_pages][Hkv][64][r_v] */
} stief_layer;

/* Paging state of the batch, shared by all layers.  block_table is [B][max_pages_per_seq] int32
 * page ids; seq_lens is [B] int32.  The library never writes either. */
typedef struct stief_batch {
  int32_t B, max_pages_per_seq;
  const int32_t* block_table;
  const int32_t* seq_lens;
} stief_batch;

/* Eq. 1 for a whole prompt: for every b, t < seq_lens[b], h: K_down[t,h,:] = rnd_bf16(K[b,t,h,:] U_k[h])
 * and the same for V, accumulated in fp32, stored to the paged pools.  K and V are bf16 with element
 * strides stride_b / v_stride_b (between sequences) and stride_t / v_stride_t (between tokens); heads are
 * contiguous blocks of 128 elements (r elements on a side without basis); rows must be 16-byte aligned.  T_max bounds seq_lens (it sizes the launch; tokens
 * beyond seq_lens[b] are never stored; the input rows of a sequence's last 128-token tile are read up
 * to T_max).
 * flags: 0, or STIEF_PREFILL_OVERLAP_PREVIOUS: the kernel may start (and write its pools) before the kernels that
 * precede it on the stream have finished, so that the per-layer launches of one prompt run without idle gaps.  The grid
 * has one CTA per SM; a CTA takes over an SM as earlier work there ends and leaves it as soon as its own tiles are
 * stored, whether or not the kernel before it is still at work, so several kernels of a run of flagged calls can be in
 * flight.  By setting the flag the caller promises that no kernel of the unbroken run of flagged calls before this one
 * (nor the unflagged call that heads it) writes this call's inputs (K, V, seq_lens, block_table, the bases) or touches
 * this layer's pools; consecutive calls for different layers satisfy that.  One CTA of the kernel waits for the
 * preceding kernel to complete before it leaves, so kernels still complete in stream order. */
#define STIEF_PREFILL_OVERLAP_PREVIOUS 1u
int stief_prefill_compress(const stief_layer* layer, const stief_batch* batch, const uint16_t* K,
                           const uint16_t* V, int64_t stride_b, int64_t stride_t, int64_t v_stride_b,
                           int64_t v_stride_t, int32_t T_max, uint32_t flags, int32_t* status, void* stream);

/* Eq. 1 for one new token per sequence: projects k_new, v_new [B][Hkv][128] and stores the rows at
 * position seq_lens[b] (the page block_table[b][seq_lens[b]/64] must already be assigned).  The
 * caller advances its seq_lens afterwards (stief_advance_seq_lens does it on the device). */
int stief_append(const stief_layer* layer, const stief_batch* batch, const uint16_t* k_new,
                 const uint16_t* v_new, int32_t* status, void* stream);

/* Eq. 1 for a run of new tokens per sequence (the cache-write half of chunked prefill, App. A.1: a later chunk of the
 * prompt is projected and stored behind what is cached already).  K, V are device bf16 [B][T_chunk][Hkv][128]
 * (r elements per head on a side without basis) with element strides as in stief_prefill_compress; chunk_lens is a
 * device int32 [B] (rows of each sequence that are real, clamped to 0 .. T_chunk) or NULL = T_chunk for all.
 *   ends_at_len = 0: row i is stored at position seq_lens[b] + i (like stief_append; advance seq_lens afterwards);
 *   ends_at_len = 1: seq_lens already counts the chunk: row i is stored at seq_lens[b] - chunk_len_b + i, the
 *                    convention of stief_mq_attention, which can follow on the same stream with the same lengths.
 * The pages of every written position must be assigned in block_table; a position outside it sets STIEF_ERR_BOUNDS.
 * Each row gets the same bits as stief_append would give it.  The whole-prompt path stays stief_prefill_compress
 * (tensor cores, HBM-bound); this one is for chunks, where the projection is a small part of the step. */
int stief_append_chunk(const stief_layer* layer, const stief_batch* batch, const uint16_t* K, const uint16_t* V,
                       int64_t stride_b, int64_t stride_t, int64_t v_stride_b, int64_t v_stride_t, int32_t T_chunk,
                       const int32_t* chunk_lens, int32_t ends_at_len, int32_t* status, void* stream);

/* Split-T planning.  The page tiles of the whole batch (one tile = 64 tokens of one KV head) are laid
 * end to end -- units (sequence, KV head, tile of up to 8 query heads) in that order -- and cut into
 * num_parts contiguous ranges of equal cost, one per CTA of a persistent kernel (cost = page tiles,
 * plus a fixed charge for every unit a range enters, which stands for the work of starting a
 * segment); a range cuts one "segment" out of every unit it overlaps and each segment yields one
 * chunk-normalised partial result.  num_parts = 0 lets the library choose (one CTA per SM of the current device, which is also
 * what stief_decode_num_parts returns); it must not exceed 65535.  The same num_parts must be given
 * to stief_decode_workspace_bytes and to every call that shares the workspace.
 * Workspace layout, n_units = B * Hkv * ceil((Hq/Hkv) / 8).  Kernels of an overlapped chain (see the flag below) may be
 * at work on one workspace at the same time, so what a kernel writes exists in four sections that consecutive fused
 * launches take in turn:
 *   control     int32 [32]                       words 0-3: per section, the epoch (a number the library gives every
 *                                                launch) of the last kernel that finished with it; words 4-7: per
 *                                                section, units finalised by the kernel now using it; zero between calls
 *   counters    int32 [4][n_units]               arrivals per unit (each section's array padded to 128 bytes); zero between calls
 *   then per section, sections at equal distances that depend on the buffer's size only (layers of different r_v share
 *   a workspace, so give every call on a buffer the same workspace_bytes):
 *   partial_o   fp32  [num_parts + n_units][8][r_v]  chunk-normalised mixes p V_down (compressed space)
 *   partial_lse fp32  [num_parts + n_units][8]       natural-log sum-exp of each segment's scores
 * A call with out == NULL (partials for stief_split_combine) always uses section 0.
 * The buffer must be 128-byte aligned and must be cleared once with stief_decode_workspace_init
 * (a cudaMemsetAsync of the whole buffer) before its first use; calls that end normally leave the
 * counters zero again.  Which section comes next is remembered per host thread and buffer address; a thread that meets
 * a buffer for the first time merely waits more than it must for a few launches.  Apart from the flagged chains below,
 * calls that share a workspace must not overlap on the GPU.  B <= 1024. */
int32_t stief_decode_num_parts(void);
size_t stief_decode_workspace_bytes(int32_t B, int32_t Hq, int32_t Hkv, int32_t r_v, int32_t num_parts);
int stief_decode_workspace_init(void* workspace, size_t workspace_bytes, void* stream);

/* Flags of the decode calls.
 * STIEF_DECODE_OVERLAP_PREVIOUS: the kernel may start before the kernels that precede it on the stream have finished
 * (programmatic dependent launch): it takes over each SM as earlier work there ends, reads its inputs, appends this
 * step's rows and streams the cache.  Before a CTA first writes the workspace it makes sure that the previous user of
 * its workspace section (four launches back) has finished, which it reads from the section's control word; it does
 * NOT wait for the kernel directly before it, so the CTAs of a short kernel that follows a long one finish, leave and
 * hand their SMs on while the long one still runs: the layers of one step, whatever their ranks, run without idle SMs
 * between them.  One CTA of every kernel (the one that finalises its last unit) waits for the preceding kernel to
 * complete before it leaves, so kernels still COMPLETE in stream order and whatever follows the chain on the stream
 * sees all of its results.
 * By setting the flag the caller promises, for every kernel of the unbroken run of flagged calls that ends directly
 * before this one (and the unflagged call that heads the run): it writes none of this call's inputs (q, k_new, v_new,
 * seq_lens, block_table, the bases, this layer's pools), does not read the cache rows this call appends, and neither
 * reads nor writes this call's out and out_lse.  Consecutive decode calls of this library on different layers, each
 * with its own output buffer, satisfy that; a call that follows stief_advance_seq_lens, or whose q is produced by the
 * preceding kernel, does not.  If the preceding stream operation is not a kernel the flag has no effect.
 * A layer may come up again within one run (a benchmark that repeats a step without advancing seq_lens): every call
 * attends to its own new token, whatever the other calls store, but which call's rows the pool keeps at that position
 * is then not defined unless all of them append the same rows.
 * The flag is honoured only when num_parts is 0 or at least the SM count; with fewer parts the launch is silently
 * serialised (same results, no overlap).  When the library cannot tell who used the section last (first launches on a
 * buffer, another host thread, a replayed graph's first nodes) the kernel falls back to waiting for the kernel
 * directly before it, which is always sufficient because of the completion order above. */
#define STIEF_DECODE_OVERLAP_PREVIOUS 1u

/* Decode attention (Eq. 18 on the reconstructions of Eq. 7, one query row per head): q [B][Hq][128]
 * bf16 attends to tokens [0, seq_lens[b] + len_add) of every sequence; len_add is 0, or 1 when the
 * token of this step was appended on the same stream and seq_lens not yet advanced.  One kernel
 * launch: query projection q U_k (the projection that compressing keys induces on queries, Sec. 2.2),
 * scores, online softmax and mix in the compressed space, and, when `out` is not NULL, the merge and
 * back-projection of stief_split_combine done by whichever CTA delivers a unit's last partial.
 * out [B][Hq][128] bf16; out_lse [B][Hq] fp32 natural-log sum-exp, optional.  A sequence of length 0
 * yields a zero row and lse = -inf.  With out == NULL only the partials are written. */
int stief_decode_attention(const stief_layer* layer, const stief_batch* batch, const uint16_t* q,
                           int32_t len_add, void* workspace, size_t workspace_bytes, int32_t num_parts,
                           uint16_t* out, float* out_lse, uint32_t flags, int32_t* status, void* stream);

/* Merge of the per-segment results by log-sum-exp (an exact re-association of Eq. 18) followed by the
 * back-projection o = o_down U_v^T (Eq. 7 applied to the mixed values; linear, so done once after the
 * merge).  Reads the workspace written by stief_decode_attention (called with out == NULL) with the
 * same batch, len_add and num_parts.  Only segments that hold tokens are read. */
int stief_split_combine(const stief_layer* layer, const stief_batch* batch, int32_t len_add,
                        const void* workspace, int32_t num_parts, uint16_t* out, float* out_lse,
                        int32_t* status, void* stream);

/* One decode step of one layer in one kernel launch: project and store (k_new, v_new) at position
 * seq_lens[b] (Eq. 1), then attend over seq_lens[b] + 1 tokens.  Same result as stief_append followed
 * by stief_decode_attention with len_add = 1. */
int stief_decode_step(const stief_layer* layer, const stief_batch* batch, const uint16_t* q,
                      const uint16_t* k_new, const uint16_t* v_new, void* workspace,
                      size_t workspace_bytes, int32_t num_parts, uint16_t* out, float* out_lse,
                      uint32_t flags, int32_t* status, void* stream);

/* The same step for callers whose activations live in host memory: q_host, k_new_host, v_new_host
 * are copied to `staging` (device, stief_host_staging_bytes) with cudaMemcpyAsync on `stream`, the
 * step runs, and out is copied back to out_host.  Nothing is synchronised: the caller waits on the
 * stream before reading out_host.  Host buffers should be pinned for the copies to be asynchronous.
 * When all four host buffers are pinned AND mapped (cudaHostAlloc / cudaHostRegister under unified
 * addressing) the copies are skipped: the kernel reads q, k_new, v_new from host memory in its prologue
 * and writes the output rows to out_host itself; `staging` is then unused. */
size_t stief_host_staging_bytes(int32_t B, int32_t Hq, int32_t Hkv);
int stief_decode_step_host(const stief_layer* layer, const stief_batch* batch, const uint16_t* q_host,
                           const uint16_t* k_new_host, const uint16_t* v_new_host, void* staging,
                           void* workspace, size_t workspace_bytes, int32_t num_parts,
                           uint16_t* out_host, uint32_t flags, int32_t* status, void* stream);

/* seq_lens[b] += delta on the device (so a captured step can be replayed). */
int stief_advance_seq_lens(int32_t* seq_lens, int32_t B, int32_t delta, void* stream);

/* stief_decode_attention for callers that cannot supply a workspace.  The paper has no counterpart:
 * this exists for integration only.  Who needs it: code that runs as a plug-in inside an engine which
 * has already claimed all device memory for its own pool and offers no allocator to plug-ins, and
 * code on a latency-critical path where cudaMalloc is ruled out because it synchronises the whole
 * device.  The split-T scratch (arrival counters and per-segment partials, same layout as the
 * workspace above) is a fixed device array of STIEF_STATIC_WORKSPACE_BYTES inside the library; every
 * GPU that loads the library holds that much memory until the process exits.  This entry point never
 * calls cudaMalloc, cudaFree or any allocating routine.
 *  - Same arguments and result as stief_decode_attention, without the workspace; `out` must not be NULL
 *    (the partials are not reachable from outside).
 *  - Limit: stief_decode_workspace_bytes(B, Hq, Hkv, r_v, num_parts) must not exceed
 *    STIEF_STATIC_WORKSPACE_BYTES, else STIEF_ERR_WORKSPACE is returned and nothing is launched
 *    (with one part per SM of a B200 and r_v = 128 that allows up to 359 (sequence, KV head) pairs
 *    of groups of at most 8 query heads).
 *  - The first call on each device looks up the array's device address (this loads the module if it
 *    is not loaded yet); make that first call outside any stream capture, with the device current.
 *  - All calls on a device share the one array and it keeps the previous call's contents.  Each call
 *    clears the counters it relies on (a cudaMemsetAsync on `stream`) before its kernel.  Two calls
 *    that overlap on the GPU -- different streams, or different host threads -- race on the array
 *    and give wrong results: serialise them. */
#define STIEF_STATIC_WORKSPACE_BYTES (8u << 20)
int stief_decode_attention_static(const stief_layer* layer, const stief_batch* batch, const uint16_t* q,
                                  int32_t len_add, int32_t num_parts, uint16_t* out, float* out_lse,
                                  int32_t* status, void* stream);

/* ---------------------------------------------------------------------------------------------------------
 * Integer-quantised compressed cache, 8-bit (stief_q8_*) and 4-bit (stief_q4_*) codes (paper Sec. 4.3: asymmetric
 * integer quantisation of the compressed cache tensors, group size 64; keys use group-wise parameters shared across
 * batch and sequence positions within a KV head, values use token-wise group parameters).
 * A group is 64 consecutive channels of the compressed dimension; the last group of ranks 32, 48 and 96 is shorter
 * (32, 48 and 32 channels).  groups(r) = ceil(r / 64).  A b-bit code c in 0 .. 2^b - 1 stands for c * scale + zero.
 * Key parameters are fixed ahead of time (calibration) per KV head and channel group and given by the caller; a key
 * outside the calibrated range is clamped.  Value parameters are computed from each row when it is written:
 * zero = min, scale = (max - min) / (2^b - 1) over the group (scale = 1 when max == min).  The quantiser sees the
 * projection K U_k / V U_v in fp32 (not rounded to bf16 first) and decides in fp32:
 * code = clamp(rint((x - zero) * (1 / scale))), ties to even.  All ranks 32, 48, 64, 96, 128; both bases must be given
 * (a side whose projection is folded into the model's linear layers is not taken: STIEF_ERR_UNSUPPORTED).
 *
 * Layout, 8-bit codes:
 *   k_codes [num_pages][Hkv][64][r_k] uint8, r fastest, indexed like the bf16 pools;
 *   v_codes [num_pages][Hkv][r_v][64] uint8, CHANNEL-major inside a page, and token t of the page sits at position
 *           pos(t) = (t & ~15) + 4*((t & 7) >> 1) + (t & 1) + 2*((t >> 3) & 1) of its channel rows (the order in which
 *           the tensor-core mix consumes tokens: raw codes are its operands, nothing is expanded in shared memory).
 * Layout, 4-bit codes (two to a byte; within every 32 consecutive indices i of a row, byte i % 16 of that block of 16
 * bytes holds index i in its low nibble when i % 32 < 16 and in its high nibble otherwise):
 *   k_codes [num_pages][Hkv][64][krow] bytes, the index being the channel; krow = r_k / 2, except r_k = 48: the row is
 *           padded to 64 nibbles, krow = 32, unused nibbles zero;
 *   v_codes [num_pages][Hkv][r_v][32] bytes, channel-major, the index being the position pos(t) above (so tokens whose
 *           positions differ by 16 inside a block of 32 share a byte).
 * Parameters, both widths: k_params [Hkv][groups(r_k)][2] fp32 (scale, zero);
 *   v_params [num_pages][Hkv][64][groups(r_v)][2] fp32 (scale, zero), token-major.
 * Alignment: code pools and v_params 128 bytes, k_params 8 bytes.  Bytes per cached (token, KV head): 8-bit
 * r_k + r_v + 8 groups(r_v); 4-bit krow + r_v / 2 + 8 groups(r_v); against 2 (r_k + r_v) for the bf16 cache.
 * Codes, bytes and nibbles of positions at or beyond a sequence's length are unspecified and never influence a result. */
typedef struct stief_qlayer {
  int32_t Hq, Hkv, d;
  int32_t r_k, r_v;
  int32_t num_pages;
  const uint16_t* U_k;
  int64_t uk_head_stride;
  const uint16_t* U_v;
  int64_t uv_head_stride;
  const float* k_params;
  uint8_t* k_codes;
  uint8_t* v_codes;
  float* v_params;
} stief_qlayer;

/* Eq. 1 for a whole prompt followed by quantisation; arguments as stief_prefill_compress. */
int stief_q8_prefill_compress(const stief_qlayer* layer, const stief_batch* batch, const uint16_t* K,
                              const uint16_t* V, int64_t stride_b, int64_t stride_t, int32_t T_max,
                              uint32_t flags, int32_t* status, void* stream);
int stief_q4_prefill_compress(const stief_qlayer* layer, const stief_batch* batch, const uint16_t* K,
                              const uint16_t* V, int64_t stride_b, int64_t stride_t, int32_t T_max,
                              uint32_t flags, int32_t* status, void* stream);

/* One new token per sequence: projects, quantises and stores k_new, v_new at position seq_lens[b]. */
int stief_q8_append(const stief_qlayer* layer, const stief_batch* batch, const uint16_t* k_new,
                    const uint16_t* v_new, int32_t* status, void* stream);
int stief_q4_append(const stief_qlayer* layer, const stief_batch* batch, const uint16_t* k_new,
                    const uint16_t* v_new, int32_t* status, void* stream);

/* Decode attention on the quantised cache: ordinary attention (Eq. 18) on the reconstructions (Eq. 7) of the
 * DEQUANTISED cache, evaluated in the compressed space (the key scale folds into the projected query, the
 * key zero-point shifts every score of a row by the same amount and so only enters out_lse).  Arguments,
 * workspace (stief_decode_workspace_bytes with the same r_v) and flags as stief_decode_attention; num_parts = 0
 * means one part per SM. */
int stief_q8_decode_attention(const stief_qlayer* layer, const stief_batch* batch, const uint16_t* q,
                              int32_t len_add, void* workspace, size_t workspace_bytes, int32_t num_parts,
                              uint16_t* out, float* out_lse, uint32_t flags, int32_t* status, void* stream);
int stief_q4_decode_attention(const stief_qlayer* layer, const stief_batch* batch, const uint16_t* q,
                              int32_t len_add, void* workspace, size_t workspace_bytes, int32_t num_parts,
                              uint16_t* out, float* out_lse, uint32_t flags, int32_t* status, void* stream);

/* One decode step of one layer on the quantised cache in one launch: project, quantise and store (k_new, v_new)
 * at position seq_lens[b], then attend over seq_lens[b] + 1 tokens.  Same result as the append call followed by the
 * attention call with len_add = 1.  With STIEF_DECODE_OVERLAP_PREVIOUS: this kernel reads its new token's codes back
 * from the pools, so a layer must not come up again within one run of flagged calls unless every such call appends
 * the same rows. */
int stief_q8_decode_step(const stief_qlayer* layer, const stief_batch* batch, const uint16_t* q, const uint16_t* k_new,
                         const uint16_t* v_new, void* workspace, size_t workspace_bytes, int32_t num_parts,
                         uint16_t* out, float* out_lse, uint32_t flags, int32_t* status, void* stream);
int stief_q4_decode_step(const stief_qlayer* layer, const stief_batch* batch, const uint16_t* q, const uint16_t* k_new,
                         const uint16_t* v_new, void* workspace, size_t workspace_bytes, int32_t num_parts,
                         uint16_t* out, float* out_lse, uint32_t flags, int32_t* status, void* stream);

/* Measurement aid (no counterpart in the paper): the next stief_decode_attention / stief_decode_step /
 * stief_decode_step_host call made by this host thread records `start_event` just before and
 * `stop_event` just after its decode kernel on the call's stream (both cudaEvent_t passed as void*),
 * so the kernel can be timed alone inside a longer step.  One-shot: cleared by that call.  Passing NULLs
 * cancels a pending request. */
int stief_time_next_decode_kernel(void* start_event, void* stop_event);

/* Measurement aid (no counterpart in the paper): the next stief_decode_attention / stief_decode_step /
 * stief_decode_step_host call made by this host thread has its kernel write, per CTA, STIEF_TRACE_SLOTS 64-bit words
 * into `trace` (device memory the caller has zeroed, 8-byte aligned, at least num_parts * STIEF_TRACE_SLOTS * 8 bytes,
 * num_parts as resolved by stief_decode_num_parts when 0; a smaller buffer switches tracing off for that call).
 * Words 0..9 are readings of the GPU's global nanosecond timer at fixed points of the CTA's life, 0 when a point was
 * never reached: 0 entry, 1 partition known, 2 first page request issued, 3 first segment's projections done,
 * 4 first page landed, 5 last page request issued, 6 last page consumed, 7 last partial stored, 8 last combine done,
 * 9 exit; words 10, 11 count the CTA's segments and the unit merges it performed; word 12 is the time at which the
 * last segment's arrival at its unit's counter was known, word 13 the SM the CTA ran on.  One-shot; NULL cancels. */
#define STIEF_TRACE_SLOTS 16
int stief_trace_next_decode_kernel(uint64_t* trace, size_t trace_bytes);

/* ---- several causal query rows per head (chunked prefill, speculative decode) --------------------------------
 * App. A.1 of the paper: during prefilling Q has one row per prefix token and Eq. 18 holds per row; the layer being
 * a decoder layer, row i of sequence b sits at absolute position p = seq_lens[b] - q_len_b + i and attends the cached
 * positions 0 .. p.  The cache must already hold the query tokens' own rows (stief_prefill_compress / stief_append
 * first), i.e. the queries are the LAST q_len_b tokens of each cached sequence.  Evaluated in the compressed space
 * like stief_decode_attention (q' = q U_k, scores and mixing on the compressed rows, one back-projection), on the
 * tcgen05 tensor cores; q' and the probabilities pass through bf16, scores, sums and the compressed output keep fp32
 * accuracy.
 *
 *   q        device, bf16 [B][n_q][Hq][d_q] with element strides q_stride_b / q_stride_t between sequences / tokens
 *            (heads and elements contiguous, strides multiples of 8); d_q = 128, or r_k when U_k is NULL (folded keys)
 *   n_q      query tokens per sequence in q and out (> 0)
 *   q_lens   device int32 [B] or NULL: how many of the n_q rows of each sequence are real (clamped to 0 .. n_q; rows
 *            beyond are neither computed nor written); NULL = n_q for every sequence.  q_len_b > seq_lens[b] sets
 *            STIEF_ERR_BOUNDS in the status word and skips the sequence
 *   out      device, bf16 [B][n_q][Hq][d_out], strides as for q; d_out = 128, or r_v when U_v is NULL (folded values:
 *            the compressed output is returned for a folded output projection)
 *   out_lse  optional device fp32 [B][n_q][Hq] (contiguous): natural-log-sum-exp of each row's scaled scores
 *   workspace, workspace_bytes, num_splits
 *            With few query rows and a long cache (speculative decode) the (sequence, KV head, 256-row) work units are too
 *            few to fill the GPU.  num_splits > 1 cuts every unit's page range into that many parts, which run as units of
 *            their own and leave partial results in `workspace` (device, 128-byte aligned, at least
 *            stief_mq_workspace_bytes(...) bytes, contents irrelevant on entry); a second small kernel merges them
 *            (log-sum-exp), normalises and back-projects.  num_splits = 1: no workspace (NULL, 0).  stief_mq_num_splits
 *            proposes a value: 1 when the units already fill the GPU, else about SMs / units, at most 32 and at most a
 *            quarter of max_pages_per_seq.  When a (sequence, KV head) has at most 128 query rows, each part is further
 *            worked through as two interleaved streams inside its CTA (the workspace size allows for that).  Too small a workspace: STIEF_ERR_WORKSPACE, nothing is launched.
 *   flags    must be 0
 * All ranks 32/48/64/96/128; Hq / Hkv must divide 128 (a 128-row tile holds whole tokens), else
 * STIEF_ERR_UNSUPPORTED.  Nothing is allocated.  Asynchronous on `stream`. */
int32_t stief_mq_num_splits(int32_t B, int32_t n_q, int32_t Hq, int32_t Hkv, int32_t max_pages_per_seq);
size_t stief_mq_workspace_bytes(int32_t B, int32_t n_q, int32_t Hq, int32_t r_v, int32_t num_splits);
int stief_mq_attention(const stief_layer* layer, const stief_batch* batch, const uint16_t* q, int64_t q_stride_b,
                       int64_t q_stride_t, int32_t n_q, const int32_t* q_lens, void* workspace, size_t workspace_bytes,
                       int32_t num_splits, uint16_t* out, int64_t out_stride_b, int64_t out_stride_t, float* out_lse,
                       uint32_t flags, int32_t* status, void* stream);

/* ---- rank selection (host only) --------------------------------------------------------------------------
 * Sequential budgeted rank selection, Algorithm 2 of the paper (Sec. 3.4, Eq. 15-17; cost c = (r_K + r_V) / (2 d_h),
 * Eq. 23): turns a target cache ratio rho into the per-layer (r_k, r_v) that stief_layer descriptors carry.  The
 * budget starts at L * rho; before layer l (0-based) the per-layer budget is what is left divided by the L - l layers
 * still to choose (the divisor of Algorithm 2); the candidate pair of least error whose cost does not exceed it is
 * taken and its cost subtracted.  Feasibility is decided in exact integer arithmetic on the bits of rho, so a pair
 * whose cost equals the budget is always accepted.  Ties in the error go to the cheaper pair, then to the smaller key
 * rank.
 *
 * All pointers are HOST pointers; nothing is launched and no CUDA call is made.
 *   cand_k[n_k], cand_v[n_v]  candidate ranks, each in 1 .. d_h, in any order (d_h itself = keep that side full rank)
 *   rho                       target ratio, 1/1024 <= rho <= 1
 *   the error tables come from exactly one of
 *     surfaces  [L][n_k][n_v] doubles, all known up front, or
 *     surface   a callback asked for layer l's table only after layers 0 .. l-1 are chosen (the paper evaluates each
 *               surface on activations that passed through the compressed prefix): it receives ctx, l, the r_k / r_v
 *               arrays (entries 0 .. l-1 valid) and writes n_k * n_v doubles row-major into delta; non-zero return
 *               aborts the selection.
 *   r_k[L], r_v[L]            outputs, owned by the caller
 *   spent                     optional: total cost sum_l c(r_k[l], r_v[l]) (never above L * rho)
 *   failed_layer              optional: -1, or the layer at which the call gave up
 * Returns STIEF_OK; STIEF_ERR_INVALID_ARG (bad sizes, both or neither table source, NaN in a table, callback
 * failure); STIEF_ERR_INFEASIBLE when no pair fits at some layer (happens exactly when rho is below the cheapest
 * candidate pair's cost, and then at layer 0). */
typedef int (*stief_surface_fn)(void* ctx, int32_t layer, const int32_t* r_k_chosen, const int32_t* r_v_chosen, double* delta);
int stief_select_ranks(int32_t L, int32_t d_h, const int32_t* cand_k, int32_t n_k, const int32_t* cand_v, int32_t n_v,
                       double rho, const double* surfaces, stief_surface_fn surface, void* ctx, int32_t* r_k,
                       int32_t* r_v, double* spent, int32_t* failed_layer);

/* Self-test of the bounded device-side waits (no counterpart in the paper).  Every wait inside the kernels -- on an
 * mbarrier that an asynchronous copy or another warp completes, on a shared counter -- polls a limited number of
 * times; when the limit is reached the CTA raises an abort flag that ends all its later waits at their next look at
 * it, writes STIEF_ERR_TIMEOUT to the status word and runs on to its normal exit (results are then meaningless, the
 * context stays healthy).  This call launches one small CTA that makes those very wait routines run out: an mbarrier
 * that nobody completes is waited on with `poll_limit` polls (1 .. 2^20), then two more waits with the kernels' own
 * limit must be cut short by the abort flag.  Nothing faults and nothing waits without limit.
 *   status  device int32, zeroed by the caller: receives STIEF_ERR_TIMEOUT
 *   report  device int32[8]: [0] first wait satisfied (expected 0), [1] its duration in SM clock cycles, [2] abort flag
 *           after it (1), [3]/[4] and [5]/[6] the same pair for the two later waits (satisfied = 0, cycles small),
 *           [7] 0x600d when the kernel reached its end
 * Asynchronous on `stream`. */
int stief_selftest_wait_limit(int32_t* status, int32_t* report, int32_t poll_limit, void* stream);

/* Measurement aid (no counterpart in the paper): one read-only pass over `bytes` (>= 16 KiB, rounded down to a multiple
 * of 16 KiB) of the 16-byte aligned device buffer `buffer`, by the decode kernels' streaming skeleton without their
 * arithmetic (one persistent CTA per SM, bulk async copies into a shared-memory ring); nothing is written.  Timed by the
 * caller with events on `stream`, it gives the bandwidth a kernel that only reads can get from the memory system, as
 * context for roofline fractions whose denominator is a copy (which reads and writes).  `status`: optional device word
 * for STIEF_ERR_TIMEOUT. */
int stief_measure_read_stream(const void* buffer, size_t bytes, int32_t* status, void* stream);

const char* stief_status_string(int status);
int stief_version(void);

#ifdef __cplusplus
}
#endif
#endif /* STIEF_H_ */
