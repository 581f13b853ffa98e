/*
 * psa.h -- C ABI of libpsa: prefix-shared attention (forward + backward) and the
 * per-response log-prob gather for DPO training, for NVIDIA B200 (sm_100a).
 *
 * Method: "Accelerating Direct Preference Optimization with Prefix Sharing"
 * (arXiv 2410.20305).  Each training sample is ONE sequence
 * [prompt | chosen | rejected]; samples are packed back to back into one row of
 * T tokens.  A query may attend to a key iff (Algorithm 3, "Prefix Sharing Mask
 * with Packing"):
 *     key index <= query index                       (causal)
 *     and both tokens belong to the same sample      (document mask)
 *     and not (query is a rejected token and key is a chosen token).
 * Algorithm 1 is the one-sample case; Algorithm 2 (the paired baseline layout)
 * is the case rejected_len = 0 with 2n samples.
 *
 * Conventions
 *   - Every function returns a psa_status_t and throws nothing.
 *   - "host" pointers are ordinary CPU memory; "device" pointers are CUDA global
 *     memory of the current device.  The library never takes ownership of a
 *     caller's buffer and never allocates tensors; it allocates only the small
 *     metadata owned by a plan.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default
 *     stream).  Kernel launches are asynchronous on that stream.
 *   - Tensor layout is token-major: element (t, h, c) of a [T, H, d] tensor is at
 *     index (t*H + h)*d + c; bf16 storage.  lse is [Hq, T] float32.
 *   - Query head h reads kv head h / (Hq / Hkv)  (grouped-query attention).
 *   - Device base pointers must be 16-byte aligned (tiles are moved by TMA).
 */
#ifndef PSA_H_
#define PSA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct psa_plan psa_plan_t; /* opaque */

typedef enum {
  PSA_OK = 0,
  PSA_ERR_INVALID_ARG = 1,          /* null pointer, negative size, bad enum, plan without device copy */
  PSA_ERR_INCONSISTENT_LENGTHS = 2, /* cu_seqlens does not match prefix+chosen+rejected */
  PSA_ERR_UNSUPPORTED = 3,          /* head_dim not in {64,128}, Hq % Hkv != 0, size over a stated maximum */
  PSA_ERR_ALIGNMENT = 4,            /* a device pointer is not 16-byte aligned */
  PSA_ERR_CUDA = 5,                 /* a CUDA runtime / driver call failed (no device, launch error, ...) */
  PSA_ERR_DEVICE_STATUS = 6,        /* psa_check_device_status: a kernel reported bad data (labels) */
  PSA_ERR_TIMEOUT = 7               /* psa_check_device_status: a bounded device-side wait expired  */
} psa_status_t;

/* Bits of the word a kernel ORs into `device_status` (device int32, may be NULL). */
#define PSA_DEVSTAT_WAIT_EXPIRED 1 /* a bounded barrier wait gave up; outputs are invalid    */
#define PSA_DEVSTAT_BAD_TARGET   2 /* dpo_logp: a scored target id was outside [0, vocab)    */
#define PSA_DEVSTAT_BAD_SEGMENT  4 /* dpo_logp: a segment id was >= n_segments               */
#define PSA_DEVSTAT_OUT_OF_BOUNDS 8 /* debug library only (libpsa_debug.so): a thread's own global
                                       index fell outside its tensor; the access was skipped     */

/* Flags of psa_plan(). */
#define PSA_PLAN_HOST_ONLY 1 /* build the tile map on the host only; no CUDA call is made */

const char* psa_status_string(psa_status_t s);

/*
 * psa_check_device_status -- turns a device status word (copied back to the host by the
 * caller, after the stream has been synchronised) into a status code: 0 -> PSA_OK;
 * PSA_DEVSTAT_WAIT_EXPIRED set -> PSA_ERR_TIMEOUT (the outputs of that call are invalid);
 * otherwise a label bit set -> PSA_ERR_DEVICE_STATUS.  Host only; no paper counterpart.
 */
psa_status_t psa_check_device_status(int32_t device_status_word);

/*
 * psa_selftest_wait_expiry -- failure-detection self test; the paper has no counterpart.
 * Launches one small CTA that waits, with the same bounded wait the attention kernels use, on
 * a barrier that nothing will ever complete.  After `limit_clocks` SM clocks (clamped to
 * [1e3, 4e9]) the wait gives up, ORs PSA_DEVSTAT_WAIT_EXPIRED into *device_status and the
 * kernel returns normally: the context stays usable.  Nothing faults, traps or spins without
 * a limit.  `spins_out` (device int64, may be NULL) receives the clocks the wait lasted.
 * Errors: INVALID_ARG (device_status NULL), CUDA.
 */
psa_status_t psa_selftest_wait_expiry(int32_t* device_status, int64_t limit_clocks, int64_t* spins_out,
                                      void* stream);

/*
 * psa_plan -- build the block-sparsity tile map of the Algorithm 3 mask once per
 * training step (Section 3.1: the sparse block mask is computed at the start of
 * every step and handed to every attention layer; fully masked blocks are
 * skipped).  One plan serves every layer and both psa_fwd and psa_bwd.
 *
 *   cu_seqlens   host int32 [n_samples+1]: first packed-row index of each sample,
 *                cu_seqlens[0] = 0, cu_seqlens[n] = T.
 *   prefix_len, chosen_len, rejected_len
 *                host int32 [n_samples]: P, C, R >= 0 per sample, with
 *                cu_seqlens[s+1] - cu_seqlens[s] = P + C + R.  Any of them may
 *                be 0 (R = 0 is plain packed causal attention).
 *   n_q_heads, n_kv_heads, head_dim
 *                Hq % Hkv == 0; head_dim 64 or 128.
 *   softmax_scale  multiplies q.k before the softmax; <= 0 selects 1/sqrt(head_dim).
 *   flags        0 or PSA_PLAN_HOST_ONLY.
 *   stream       the upload of the tile map is enqueued here (ignored if HOST_ONLY).
 *   out          receives the plan; destroy with psa_plan_destroy.
 *
 * Tiles are 128 x 128 and aligned to the start of each sample.  A (query tile,
 * key tile) pair is dropped when every pair in it is masked, marked FULL when
 * none is, and PARTIAL otherwise (masked per element in registers).
 * Errors: INVALID_ARG, INCONSISTENT_LENGTHS, UNSUPPORTED, CUDA.
 */
psa_status_t psa_plan(const int32_t* cu_seqlens, const int32_t* prefix_len,
                      const int32_t* chosen_len, const int32_t* rejected_len,
                      int32_t n_samples, int32_t n_q_heads, int32_t n_kv_heads,
                      int32_t head_dim, float softmax_scale, int32_t flags,
                      void* stream, psa_plan_t** out);

/*
 * Copies a HOST_ONLY plan's tile map to the current device (no-op if already there).  The copy is
 * asynchronous on `stream` (from a pinned staging buffer owned by the library).  Calls that use the
 * plan on another stream make that stream wait for the copy themselves.
 */
psa_status_t psa_plan_upload(psa_plan_t* plan, void* stream);

/*
 * Frees the plan's host metadata and returns its device metadata (a few hundred KB) to a small
 * cache inside the library, from which the next plan takes it: building a plan per step costs no
 * cudaMalloc / cudaFree and does not wait for the device.  The call does not wait either: work that
 * was enqueued with the plan may still be running; the library orders the next owner's upload
 * behind it.  The streams the plan was used on must still exist.  NULL is accepted.
 */
psa_status_t psa_plan_destroy(psa_plan_t* plan);

/*
 * psa_plan_stats -- any output pointer may be NULL.
 *   total_tokens        T
 *   useful_pairs        unmasked (q, kv) pairs per query head
 *   live_tiles          (query tile, key tile) pairs kept in the map
 *   partial_tiles       how many of those need per-element masking in the forward
 *   bwd_workspace_bytes size of the device scratch buffer psa_bwd needs
 */
psa_status_t psa_plan_stats(const psa_plan_t* plan, int64_t* total_tokens,
                            int64_t* useful_pairs, int64_t* live_tiles,
                            int64_t* partial_tiles, size_t* bwd_workspace_bytes);

/*
 * psa_plan_counts / psa_plan_export -- read the tile map back (tests, tools).
 * direction 0 = forward map (one record per query tile, entries = key tiles),
 * direction 1 = transposed map for the backward (one record per key tile,
 * entries = query tiles).
 * A record is 8 int32: { row0, sample_start, local0, sample_len, chosen_start,
 * rejected_start, entry_offset, entry_count }, where row0 is the packed-row
 * index of the tile's first row, local0 = row0 - sample_start, and
 * chosen_start / rejected_start are relative to sample_start.  An entry is
 * (tile_index_within_sample << 2) | (precise << 1) | needs_mask, where `precise`
 * marks query tiles holding a row with fewer than 128 visible keys: for those the
 * kernels keep the probabilities (and dS) as a sum of two bf16 terms.
 * `tiles` is host int32 [n_tiles*8], `entries` host int32 [n_entries].
 */
psa_status_t psa_plan_counts(const psa_plan_t* plan, int32_t direction,
                             int32_t* n_tiles, int32_t* n_entries);
psa_status_t psa_plan_export(const psa_plan_t* plan, int32_t direction,
                             int32_t* tiles, int32_t* entries);

/*
 * psa_fwd -- attention forward under the plan's mask (Section 3.1).
 *   S = scale * Q K^T on the live tiles, softmax over the allowed keys of each
 *   row in fp32, O = P V;  lse[h][t] = log sum_j exp(S[t][j])  (natural log).
 *   q        device bf16 [T, Hq, d]        k, v   device bf16 [T, Hkv, d]
 *   o        device bf16 [T, Hq, d] (out)  lse    device fp32 [Hq, T] (out)
 *   device_status  device int32 or NULL; bits are ORed in, never cleared.
 * Rows >= T are neither read nor written.  T = 0 is a no-op.
 * Errors: INVALID_ARG (also: the plan was uploaded on another device than the current one),
 * ALIGNMENT, CUDA.
 */
psa_status_t psa_fwd(const psa_plan_t* plan, const void* q, const void* k, const void* v,
                     void* o, float* lse, int32_t* device_status, void* stream);

/*
 * psa_bwd -- exact gradient of psa_fwd; probabilities are recomputed from lse.
 *   D_i = dO_i . O_i;  P = exp(S - lse);  dV = P^T dO;  dP = dO V^T;
 *   dS = P * (dP - D);  dQ = scale * dS K;  dK = scale * dS^T Q;
 *   dK and dV are summed over the Hq/Hkv query heads of each kv head.
 *   d_o, q, o   device bf16 [T, Hq, d]     k, v    device bf16 [T, Hkv, d]
 *   lse         device fp32 [Hq, T] as written by psa_fwd
 *   dq          device bf16 [T, Hq, d] (out)   dk, dv  device bf16 [T, Hkv, d] (out)
 *   workspace   device scratch of psa_plan_stats().bwd_workspace_bytes bytes,
 *               256-byte aligned; contents on entry are ignored, on exit undefined.
 * The call is stateless: the same plan may serve any number of layers.
 * Errors: INVALID_ARG, ALIGNMENT, CUDA.
 */
psa_status_t psa_bwd(const psa_plan_t* plan, const void* d_o, const void* q, const void* k,
                     const void* v, const void* o, const float* lse,
                     void* dq, void* dk, void* dv, void* workspace,
                     int32_t* device_status, void* stream);

/*
 * psa_selftest_bounds -- self test of the debug library's checked indices; the paper has no
 * counterpart.  Tiles move by TMA, which clips every box to its tensor; the indices that threads
 * form themselves (lse / delta words, ragged last tiles, fp32 gradient rows) are checked in
 * libpsa_debug.so (the same sources built with -DPSA_DEBUG_BOUNDS): an index outside its tensor
 * sets PSA_DEVSTAT_OUT_OF_BOUNDS and the access is skipped.  This call runs one index inside and
 * one outside a 4-element tensor through that check: in the debug library *result = 1 and the bit
 * is set; in the product library, where the check compiles to nothing, *result = 3 and no bit.
 *   device_status, result   device int32 [1]
 * Errors: INVALID_ARG, CUDA.
 */
psa_status_t psa_selftest_bounds(int32_t* device_status, int32_t* result, void* stream);

/*
 * psa_bwd_f32 -- psa_bwd with fp32 gradient outputs (same computation, same kernels; the only
 * difference is that the fp32 accumulators are written out as they are instead of being rounded
 * to bf16).  For callers that accumulate gradients in fp32, and for checking the gradients
 * against a reference without the bf16 output rounding in the way.
 *   dq          device fp32 [T, Hq, d] (out): serves as the accumulator itself
 *   dk, dv      device fp32 [T, Hkv, d] (out)
 *   workspace   as for psa_bwd (same size; only its delta part is used)
 *   everything else as for psa_bwd.
 * Errors: INVALID_ARG, ALIGNMENT, CUDA.
 */
psa_status_t psa_bwd_f32(const psa_plan_t* plan, const void* d_o, const void* q, const void* k,
                         const void* v, const void* o, const float* lse,
                         float* dq, float* dk, float* dv, void* workspace,
                         int32_t* device_status, void* stream);

/*
 * psa_bwd_static_scratch -- psa_bwd without the workspace argument.  The paper has no
 * counterpart; this entry point exists for callers that have no way to provide scratch
 * memory at the time of the call: for example a step function running after the
 * framework's caching allocator has taken the whole device (a raw cudaMalloc from a
 * library would fail or fragment it), or a latency-critical loop that must not trigger
 * the device-wide synchronisation that cudaMalloc / cudaFree imply.
 *
 * The call allocates nothing: no cudaMalloc, no cudaFree, no allocating library routine.
 * Its scratch (the fp32 dq accumulator and the delta vector) is a fixed array of
 * PSA_STATIC_SCRATCH_BYTES (32 MiB) inside the library's device image; every GPU that
 * loads the library holds that array until the process exits.
 *
 *   Arguments   as psa_bwd, minus `workspace`.  Inputs and outputs are still the caller's.
 *   Limit       plans with psa_plan_stats().bwd_workspace_bytes > PSA_STATIC_SCRATCH_BYTES
 *               (roughly T * Hq * d > 8.3 M elements, e.g. more than 2030 tokens at 32
 *               heads of 128) are rejected with PSA_ERR_UNSUPPORTED before anything is
 *               launched; with PSA_DEBUG set in the environment the sizes are printed.
 *   First call  the first call on each device looks up the array's device address (with
 *               that device current) and keeps it.  Make that first call before any stream
 *               capture begins on the device.
 *   Sharing     all calls on a device use the same array, which keeps the previous call's
 *               contents.  The call itself clears the part that must start at zero (the dq
 *               accumulator) and overwrites the rest before reading it, so calls that run
 *               one after another are independent.  Two calls that overlap on the GPU
 *               (different streams, or different host threads) race on the array and give
 *               wrong gradients: serialise them.
 * Errors: INVALID_ARG, ALIGNMENT, UNSUPPORTED (too large), CUDA.
 */
#define PSA_STATIC_SCRATCH_BYTES (32u * 1024u * 1024u)
psa_status_t psa_bwd_static_scratch(const psa_plan_t* plan, const void* d_o, const void* q,
                                    const void* k, const void* v, const void* o, const float* lse,
                                    void* dq, void* dk, void* dv, int32_t* device_status,
                                    void* stream);

/*
 * psa_step_host -- one forward and one backward pass of the attention (Algorithm 3; the
 * two calls above) on HOST buffers.  The call enqueues on `stream`, in this order: the
 * copies of q, k, v, d_o from host memory into the arena, psa_fwd, psa_bwd, and the copies
 * of o, lse, dq, dk, dv back to host memory.  It does not synchronise: the outputs are valid
 * once the stream has reached the end of the call's work.  Calls on different streams with
 * different arenas overlap (one call's copies with another's kernels).
 *   h_q, h_do   host bf16 [T, Hq, d]       h_k, h_v    host bf16 [T, Hkv, d]      (in)
 *   h_o, h_dq   host bf16 [T, Hq, d]       h_dk, h_dv  host bf16 [T, Hkv, d]      (out)
 *   h_lse       host fp32 [Hq, T]                                                (out)
 *               Pinned (page-locked) host memory makes the copies asynchronous; pageable
 *               memory works but serialises them with the host.
 *   arena       device memory of at least psa_step_host_arena_bytes(plan) bytes, 256-byte
 *               aligned, owned by the caller; it holds the device copies of every tensor
 *               and the backward scratch.  Contents on entry are ignored, on exit undefined.
 *               The call allocates nothing.
 * Errors: INVALID_ARG (null pointer, arena too small), ALIGNMENT, CUDA.
 */
size_t psa_step_host_arena_bytes(const psa_plan_t* plan);
psa_status_t psa_step_host(const psa_plan_t* plan, const void* h_q, const void* h_k, const void* h_v,
                           const void* h_do, void* h_o, float* h_lse, void* h_dq, void* h_dk,
                           void* h_dv, void* arena, size_t arena_bytes, int32_t* device_status,
                           void* stream);

/*
 * dpo_logp -- summed log-probabilities per response (Section 2.1: the total
 * log probability of each completion; Section 3.2: responses are recovered at
 * loss time from their boundaries).
 *   out[g] = sum over scored (row t, label y) with response id g of
 *            logits[t][y] - log sum_v exp(logits[t][v])
 *   logits        device [n_rows, vocab], row stride `row_stride` elements
 *   logits_dtype  PSA_DTYPE_F32 or PSA_DTYPE_BF16
 *   targets       device int32 [n_rows]: label scored by row t
 *   segment_ids   device int32 [n_rows]: response id of that label, or < 0 if the
 *                 row scores nothing through this array (its logits are then not
 *                 read unless a fork names the row)
 *   fork_rows, fork_targets, fork_segments
 *                 device int32 [n_forks] (may be NULL when n_forks = 0): rows that
 *                 score a SECOND label.  In the shared layout the last prompt row
 *                 predicts both the first chosen and the first rejected token.
 *   out           device fp32 [n_segments], overwritten
 *   device_status device int32 or NULL: PSA_DEVSTAT_BAD_TARGET / BAD_SEGMENT are
 *                 ORed in and the offending label is skipped; nothing faults.
 * Accumulation is fp32; the order of the per-row additions into out[] is not fixed.
 * Errors: INVALID_ARG, ALIGNMENT (rows must start 16-byte aligned), CUDA.
 */
#define PSA_DTYPE_F32 0
#define PSA_DTYPE_BF16 1
psa_status_t dpo_logp(const void* logits, int32_t logits_dtype, int64_t n_rows, int64_t vocab,
                      int64_t row_stride, const int32_t* targets, const int32_t* segment_ids,
                      const int32_t* fork_rows, const int32_t* fork_targets,
                      const int32_t* fork_segments, int32_t n_forks, int32_t n_segments,
                      float* out, int32_t* device_status, void* stream);

/*
 * psa_position_ids -- position ids of the shared layout (Section 3.1: the positions are set so
 * that the sequences are the same as in the paired format): prompt and chosen tokens count on
 * from 0 at the sample start, the j-th rejected token gets P + j.  Host only.
 *   cu_seqlens, prefix_len, chosen_len, rejected_len, n_samples   as for psa_plan
 *   position_ids   host int32 [T] (out)
 * Errors: INVALID_ARG, INCONSISTENT_LENGTHS.
 */
psa_status_t psa_position_ids(const int32_t* cu_seqlens, const int32_t* prefix_len,
                              const int32_t* chosen_len, const int32_t* rejected_len,
                              int32_t n_samples, int32_t* position_ids);

/*
 * psa_rope -- rotary position embedding of a [n_tokens, n_heads, head_dim] bf16 tensor with
 * per-token position ids, "rotate-half" convention (Llama family): with x = [x1 | x2] split at
 * head_dim / 2 and angle_i = pos * rope_theta^(-2i / head_dim),
 *     y1 = x1 cos - x2 sin,   y2 = x2 cos + x1 sin.
 * q and k are rotated with it before psa_fwd (the kernels themselves are position-free).
 *   x, y           device bf16; y may be x (in place)
 *   position_ids   device int32 [n_tokens]
 *   head_dim       multiple of 16, at most 256
 * Errors: INVALID_ARG, UNSUPPORTED, ALIGNMENT, CUDA.
 */
psa_status_t psa_rope(const void* x, void* y, const int32_t* position_ids, int64_t n_tokens,
                      int32_t n_heads, int32_t head_dim, float rope_theta, void* stream);

/*
 * psa_pack_ffd -- first-fit-decreasing packing of prefix-shared units into rows of a fixed
 * packing length (Section 3.2: the packing unit is the shared prompt with both responses;
 * Section 4.3.2: a first-fit-decreasing sampler, packing length = batch size x max unit length).
 * Host only, no CUDA call.
 *   unit_len      host int32 [n_units]: P + C + R of each sample (for the paired baseline layout
 *                 pass 2P + C + R)
 *   capacity      the packing length
 *   bin_of_unit   host int32 [n_units] (out): index of the pack each unit goes to.  Units are
 *                 taken from the longest to the shortest (ties: lower index first) and placed
 *                 into the first pack, in order of creation, that still has room.
 *   n_bins        host int32 (out): number of packs opened
 * Errors: INVALID_ARG (null pointer, negative length, capacity <= 0), UNSUPPORTED (a unit is
 * longer than the capacity; nothing is written).
 */
psa_status_t psa_pack_ffd(const int32_t* unit_len, int32_t n_units, int32_t capacity,
                          int32_t* bin_of_unit, int32_t* n_bins);

/*
 * psa_pack_ffd_emit -- psa_pack_ffd followed by the lay-out of every pack in the form psa_plan
 * takes (Section 3.2: the prompt and its two responses are packed as one unit; Section 4.3.2).
 * Host only, no CUDA call.
 *   prefix_len, chosen_len, rejected_len   host int32 [n_units]: P, C, R of each sample
 *   capacity     the packing length
 *   paired       0: shared layout, one sample (P, C, R) of P + C + R tokens per unit;
 *                1: the unshared baseline layout, two samples (P, C, 0) and (P, R, 0) per unit,
 *                   kept next to each other in one pack (unit length 2P + C + R)
 *   bin_of_unit  host int32 [n_units] (out): the pack of each unit, as psa_pack_ffd
 *   n_packs      host int32 (out)
 *   pack_sample_offset   host int32 [n_units + 1] (out; n_packs + 1 entries written): the samples
 *                of pack b are entries [off[b], off[b+1]) of the four arrays below
 *   sample_unit  host int32 [m] (out), m = n_units (shared) or 2 n_units (paired): the unit a
 *                sample came from.  Within a pack the units stand in the order the packer placed
 *                them (longest first, ties by index).
 *   out_prefix_len, out_chosen_len, out_rejected_len   host int32 [m] (out)
 *   out_cu_seqlens   host int32 [m + n_units] (out): the packs' cu_seqlens arrays one after the
 *                other; pack b's array starts at index off[b] + b and has off[b+1] - off[b] + 1
 *                entries, the first of them 0.
 * Pack b is planned with
 *   psa_plan(out_cu_seqlens + off[b] + b, out_prefix_len + off[b], out_chosen_len + off[b],
 *            out_rejected_len + off[b], off[b+1] - off[b], ...).
 * Errors: INVALID_ARG, UNSUPPORTED (a unit is longer than the capacity; nothing is written).
 */
psa_status_t psa_pack_ffd_emit(const int32_t* prefix_len, const int32_t* chosen_len,
                               const int32_t* rejected_len, int32_t n_units, int32_t capacity,
                               int32_t paired, int32_t* bin_of_unit, int32_t* n_packs,
                               int32_t* pack_sample_offset, int32_t* sample_unit,
                               int32_t* out_prefix_len, int32_t* out_chosen_len,
                               int32_t* out_rejected_len, int32_t* out_cu_seqlens);

/*
 * psa_logp_labels -- which logits row scores which token on the shared layout, for dpo_logp
 * (Section 2.1: the log-probs are those of the paired format; Section 3.2: responses are
 * recovered from their boundaries).  The paper gives no formula; the reading is next-token
 * scoring inside each response's own context: row t scores token t + 1 of the same response;
 * the last prompt row scores BOTH the first chosen and the first rejected token (the second of
 * the two labels goes to the fork list); the last chosen and the last rejected row score nothing;
 * with an empty prompt the first token of a response has no scoring row.  Host only.
 *   token_ids    host int32 [T]: the packed row's tokens
 *   cu_seqlens, prefix_len, chosen_len, rejected_len, n_samples   as for psa_plan
 *   targets, segment_ids   host int32 [T] (out): label and response id (2s chosen, 2s+1
 *                rejected, -1 none) of each row, as dpo_logp takes them
 *   fork_rows, fork_targets, fork_segments   host int32 [n_samples] (out; n_forks entries written)
 *   n_forks      host int32 (out)
 * Errors: INVALID_ARG, INCONSISTENT_LENGTHS.
 */
psa_status_t psa_logp_labels(const int32_t* token_ids, const int32_t* cu_seqlens,
                             const int32_t* prefix_len, const int32_t* chosen_len,
                             const int32_t* rejected_len, int32_t n_samples, int32_t* targets,
                             int32_t* segment_ids, int32_t* fork_rows, int32_t* fork_targets,
                             int32_t* fork_segments, int32_t* n_forks);

/*
 * dpo_loss -- the DPO loss of Eq. 1 (Section 2.1) from the four summed log-probs per sample.
 * The equation is printed as a ratio of logs; it is read as
 *     loss = mean over samples s of  -log sigmoid(beta * margin_s),
 *     margin_s = (policy[2s] - ref[2s]) - (policy[2s+1] - ref[2s+1])     (2s = chosen, 2s+1 = rejected).
 *   policy_logps, ref_logps  device fp32 [2 * n_samples], as written by dpo_logp for the policy and
 *                            the reference model
 *   loss                     device fp32 [1] (out)
 *   coef                     device fp32 [2 * n_samples] (out): d loss / d policy_logps
 * Errors: INVALID_ARG, CUDA.
 */
psa_status_t dpo_loss(const float* policy_logps, const float* ref_logps, int32_t n_samples, float beta,
                      float* loss, float* coef, void* stream);

/*
 * simpo_loss -- the length-normalised, reference-free paired loss (SimPO; Section 1 names it
 * beside DPO as a paired-preference method that the shared layout serves):
 *     loss = mean over samples s of
 *            -log sigmoid(beta * (policy[2s] / len[2s] - policy[2s+1] / len[2s+1]) - gamma).
 *   policy_logps  device fp32 [2 * n_samples], as written by dpo_logp
 *   lengths       device int32 [2 * n_samples]: scored tokens of each response (all >= 1)
 *   loss          device fp32 [1] (out)
 *   coef          device fp32 [2 * n_samples] (out): d loss / d policy_logps, ready for dpo_logp_bwd
 * Errors: INVALID_ARG, CUDA.  A length < 1 sets PSA_DEVSTAT_BAD_SEGMENT in device_status (may be
 * NULL) and that sample contributes nothing.
 */
psa_status_t simpo_loss(const float* policy_logps, const int32_t* lengths, int32_t n_samples, float beta,
                        float gamma, float* loss, float* coef, int32_t* device_status, void* stream);

/*
 * orpo_loss -- the odds-ratio paired loss (ORPO; Section 1 names it beside DPO and SimPO): with
 * a_g = policy[g] / len[g], P_g = exp(a_g) and lo_g = a_g - log(1 - P_g),
 *     loss = mean over samples s of  -a_{2s} + lambda * -log sigmoid(lo_{2s} - lo_{2s+1}).
 *   policy_logps, lengths, loss, coef, device_status   as for simpo_loss
 * Errors: INVALID_ARG, CUDA.  A length < 1 sets PSA_DEVSTAT_BAD_SEGMENT and that sample contributes
 * nothing.  A mean log-prob of exactly 0 (probability 1) makes the odds infinite, as in the definition.
 */
psa_status_t orpo_loss(const float* policy_logps, const int32_t* lengths, int32_t n_samples, float lambda,
                       float* loss, float* coef, int32_t* device_status, void* stream);

/*
 * dpo_logp_bwd -- gradient of  sum_g coef[g] * out[g]  (out as written by dpo_logp) with respect
 * to the logits:  dlogits[t][v] = sum over the labels (t, y, g) scored by row t of
 *                 coef[g] * (1[v == y] - softmax(logits[t])[v]).
 * Rows that score nothing are written as zeros and their logits are not read.
 *   logits .. n_segments   exactly as for dpo_logp
 *   coef                   device fp32 [n_segments], e.g. from dpo_loss
 *   dlogits                device, same dtype, shape and row stride as logits (out); must not
 *                          alias logits
 *   device_status          as for dpo_logp; invalid labels are reported and skipped
 * A row may carry at most 4 labels (its own and up to 3 forks); further ones are ignored.
 * Errors: INVALID_ARG, ALIGNMENT, UNSUPPORTED, CUDA.
 */
psa_status_t dpo_logp_bwd(const void* logits, int32_t logits_dtype, int64_t n_rows, int64_t vocab,
                          int64_t row_stride, const int32_t* targets, const int32_t* segment_ids,
                          const int32_t* fork_rows, const int32_t* fork_targets,
                          const int32_t* fork_segments, int32_t n_forks, int32_t n_segments,
                          const float* coef, void* dlogits, int32_t* device_status, void* stream);

/*
 * psa_profile_events -- measurement aid, no counterpart in the paper.  Registers a
 * pair of cudaEvent_t (passed as void*) that the next calls record on their stream
 * immediately before and after one chosen kernel, so that a benchmark can time that
 * kernel alone while it runs inside a whole step.
 *   which   0 = the psa_fwd kernel, 1 = the main psa_bwd kernel (without its helpers),
 *           2 = the dpo_logp kernel, 3 = psa_bwd's first helper (delta, and the clearing of
 *           the dq accumulator), 4 = psa_bwd's last helper (dq accumulator -> bf16)
 *   start, stop   events created with timing enabled; pass NULL, NULL to unregister.
 * Process-global and not thread-safe; the events must outlive the calls they time.
 * Errors: INVALID_ARG (bad `which`, or only one of the two events given).
 */
psa_status_t psa_profile_events(int32_t which, void* start, void* stop);

#ifdef __cplusplus
}
#endif
#endif /* PSA_H_ */
