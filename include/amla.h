/*
 * libamla -- paged MLA decode attention with exponent-add output rescaling (sm_100a).
 *
 * C ABI.  All pointers are borrowed; the library allocates no device memory and
 * keeps no state between calls beyond a per-device cache of device attributes.  Work is enqueued on the caller's stream with no
 * host synchronisation (sequence lengths are never read on the host).  Functions
 * return an amla_status; nothing throws, aborts or prints.
 *
 * Shapes are those of the paper's decode setting (Section 3.1: G query rows of
 * width D_k = 576 against a latent cache whose rows serve as K (576 columns) and,
 * through their first D_v = 512 columns, as V; Section 2.2).  Paging, per-sequence
 * lengths, the lse output, the causal rule between speculative query tokens and
 * split-KV are additions the paper does not describe; they are defined below.
 */
#ifndef AMLA_H_
#define AMLA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  AMLA_OK = 0,
  AMLA_ERR_INVALID_ARG = -1,    /* null pointer, non-positive size, misaligned buffer   */
  AMLA_ERR_UNSUPPORTED = -2,    /* shape or device outside what the kernels cover       */
  AMLA_ERR_WORKSPACE = -3,      /* workspace smaller than amla_mla_decode_workspace_size */
  AMLA_ERR_CUDA = -4,           /* a CUDA runtime/driver call failed                    */
  AMLA_ERR_DEVICE_TIMEOUT = -5, /* a bounded device-side wait ran out (see amla_check_status) */
  AMLA_ERR_STATIC_LIMIT = -6    /* amla_mla_decode_static: problem or device beyond its built-in scratch */
} amla_status;

/* Rescale variants, for A/B measurements (flags argument of amla_mla_decode_ex).
 *   AMLA_RESCALE_ALG2 : Algorithm 2 as specified: P scaled by S16 = bf16(1/r_i), the accumulator
 *                       updated by one INT32 add of N = dn*2^23 + round(2^23*(1.5*(c_i/c_{i-1}-1)+1e-6))
 *                       (Lemma 3.1 + Appendix A).  Default.
 *   AMLA_RESCALE_FOLD : Eq. 3 with 1/r_i folded exactly into the exponential's argument: the add is a
 *                       pure exponent add dn*2^23 and is needed only when n_i changes.
 *   AMLA_RESCALE_FMUL : Algorithm 1's FP32 multiply by exp(m_{i-1}-m_i) (the baseline the paper replaces).
 * AMLA_FLAG_UNGUARDED_ADD uses the literal single integer add of Algorithm 2 line 14 (corrupts
 * accumulators that are exactly 0.0 or below 2^-97; measurement only).
 *
 * AMLA_LAZY(tau), tau = 0..15 octaves: how far a tile's maximum may exceed the reference that P, l and
 * the accumulator are expressed against before the reference is moved (and the accumulator rescaled).
 * tau = 0 moves it with every new running maximum, which is Algorithm 2 to the letter.  With tau > 0
 * the probabilities may reach 2^tau instead of 1 between moves -- harmless in bf16 P and FP32
 * accumulators -- and rescales become rare; lines 6-12 of Algorithm 2 then run at the moves only.
 * amla_mla_decode uses AMLA_RESCALE_ALG2 | AMLA_LAZY(AMLA_DEFAULT_TAU).
 */
enum {
  AMLA_RESCALE_ALG2 = 0,
  AMLA_RESCALE_FOLD = 1,
  AMLA_RESCALE_FMUL = 2,
  AMLA_RESCALE_MASK = 3,
  AMLA_FLAG_UNGUARDED_ADD = 4,
  AMLA_FLAG_KERNEL_SIMT = 8,    /* run the scalar bring-up kernel instead of the tensor-core kernels */
  AMLA_FLAG_KERNEL_ROWS128 = 16, /* A/B measurements: treat sequences with more than 128 query rows as independent
                                    128-row blocks (each streams the cache on its own) instead of running the
                                    256-row kernel, in which one load of a cache tile serves all 256 rows */
  AMLA_LAZY_SHIFT = 8,
  AMLA_LAZY_MASK = 0xF00,
  AMLA_DEFAULT_TAU = 8
};
#define AMLA_LAZY(tau) (((tau) & 0xF) << 8)

/* Human-readable name of a status code (static storage). */
const char* amla_status_string(int status);

/* Bytes of device workspace amla_mla_decode needs for these sizes on `device`
 * (its SM count bounds the number of KV splits).  Host-only; no CUDA work is enqueued. */
int amla_mla_decode_workspace_size(int B, int Sq, int H, int max_blocks_per_seq, int device,
                                   size_t* bytes_out);

/*
 * out[b,t,h,:] = softmax_j(scale * q[b,t,h,:] . k_j) @ k_j[0:512]   over the visible keys j of sequence b,
 * lse[b,t,h]   = ln sum_j exp(scale * q[b,t,h,:] . k_j)                          (Eq. 1; Algorithm 2)
 *
 * Key j of sequence b is row (j % 64) of page block_table[b][j / 64] of kv_cache.  Query token t sees
 * key j iff 0 <= j < seqlens[b] and j <= seqlens[b] - Sq + t (the Sq query tokens are the last Sq
 * positions; each sees itself and everything before).  A row with no visible key gets out = 0,
 * lse = -inf.
 *
 *   q            device, bf16 [B, Sq, H, 576], contiguous, 16-byte aligned
 *   kv_cache     device, bf16 [num_blocks, 64, 576], contiguous, 16-byte aligned.  Rows of a used page
 *                beyond the sequence length must hold finite values (they are multiplied by zero).
 *   block_table  device, int32 [B, max_blocks_per_seq]; entries beyond ceil(seqlens[b]/64) are ignored
 *   seqlens      device, int32 [B], 0 <= seqlens[b] <= 64 * max_blocks_per_seq
 *                (read while the kernel in front on the stream may still be draining if that kernel is one of
 *                this library's own, which never write it; a caller's kernel that produces seqlens must not itself
 *                release its dependents early by programmatic dependent launch)
 *   out          device, bf16 [B, Sq, H, 512], 16-byte aligned
 *   lse          device, fp32 [B, Sq, H], natural logarithm
 *   workspace    device, 256-byte aligned, at least amla_mla_decode_workspace_size() bytes; contents
 *                need not be preserved or initialised; calls that overlap in time need distinct ones
 *   cuda_stream  a cudaStream_t (NULL = default stream)
 *
 * Supported: 1 <= Sq <= 8, 1 <= H <= 128 (any Sq*H up to 1024 query rows per sequence; up to 128 rows are
 * processed as one block by a pair of SMs, more than 128 rows in blocks of 256 by four SMs that share every
 * cache tile they load); page size 64; sm_100 devices only (AMLA_ERR_UNSUPPORTED otherwise).
 * Argument errors are reported before anything is launched.
 */
int amla_mla_decode(const void* q, const void* kv_cache, const int32_t* block_table,
                    const int32_t* seqlens, float softmax_scale, int B, int Sq, int H, int num_blocks,
                    int max_blocks_per_seq, void* out, float* lse, void* workspace,
                    size_t workspace_bytes, void* cuda_stream);

/*
 * amla_mla_decode without a workspace argument, for callers that cannot allocate device memory.
 * (The paper has no counterpart; this is a packaging variant of the call above.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- a serving loop that must never enter the
 * allocator on its hot path, a process whose device memory was carved up completely at start-up, a plugin that
 * is handed input and output buffers and nothing else.  The scratch the decode needs (schedule prefix, status
 * word, FP32 partials of split sequences) lives in a fixed array inside the library image instead: about 37 MiB
 * that every GPU which loads the library holds until the process exits.  The call itself performs no cudaMalloc,
 * cudaFree or any other allocating call.
 *
 * Arguments, layouts, the visibility rule and the results are those of amla_mla_decode (default rescale variant).
 * Limits: B * ceil(Sq*H/128) <= AMLA_STATIC_MAX_ITEMS and a device with at most AMLA_STATIC_MAX_SMS SMs; beyond
 * either the call returns AMLA_ERR_STATIC_LIMIT and launches nothing.
 *
 * The first call on a device looks up the device address of the array (a one-time query, made with that device
 * current); make that first call before any stream capture begins.  All calls on a device share the one array and
 * it keeps the previous call's contents: that is harmless, because each call rewrites everything it later reads,
 * but two calls whose kernels overlap on the GPU (different streams, no ordering between them) race on it and
 * give undefined results.  Order such calls, or use amla_mla_decode with one workspace per stream.
 * The bounded-wait status word is inside the array: read it with amla_static_check_status, not amla_check_status.
 */
#define AMLA_STATIC_MAX_ITEMS 4096
#define AMLA_STATIC_MAX_SMS 148
int amla_mla_decode_static(const void* q, const void* kv_cache, const int32_t* block_table,
                           const int32_t* seqlens, float softmax_scale, int B, int Sq, int H, int num_blocks,
                           int max_blocks_per_seq, void* out, float* lse, void* cuda_stream);

/* amla_check_status for amla_mla_decode_static: synchronises `cuda_stream` and reads the status word that the
 * kernels keep in the built-in scratch of the current device.  AMLA_OK, or AMLA_ERR_DEVICE_TIMEOUT if a bounded
 * wait expired during the last static call (its outputs are then undefined).  Allocates nothing. */
int amla_static_check_status(void* cuda_stream);

/* Same as amla_mla_decode, with a flags word selecting a rescale variant (see the enum above). */
int amla_mla_decode_ex(const void* q, const void* kv_cache, const int32_t* block_table,
                       const int32_t* seqlens, float softmax_scale, int B, int Sq, int H,
                       int num_blocks, int max_blocks_per_seq, void* out, float* lse, void* workspace,
                       size_t workspace_bytes, void* cuda_stream, int flags);

/*
 * The same decode on an FP8 cache (the remark after Lemma 3.1: the rescaling trick is tied to the accumulator's
 * format, not to the inputs'; the accumulator stays FP32, Q and P~ stay bf16).
 *
 *   kv_cache_e4m3  device, uint8 [num_blocks, 64, 576], 16-byte aligned: OCP FP8 E4M3 (1 sign, 4 exponent bits with
 *                  bias 7, 3 mantissa bits; no infinities, S.1111.111 is NaN).  The value of an element is
 *                  decode(byte) * kv_scale; its first 512 columns are V.  Page layout and block table as above.
 *   kv_scale       one dequantisation factor for the whole cache
 *   workspace      at least amla_mla_decode_fp8_workspace_size() bytes, 256-byte aligned
 *   flags          as for amla_mla_decode_ex
 *
 * Two passes: the pages the batch uses are first widened, exactly, into a bf16 copy inside the workspace
 * (B * max_blocks_per_seq pages of 73 728 bytes), kv_scale is folded into the softmax scale and into the final
 * normalisation, and the bf16 kernels run on the copy.  The FP8 cache saves device memory, not traffic: a call reads
 * the FP8 pages and writes and reads their copy.  Everything else (visibility rule, outputs, errors) is as for
 * amla_mla_decode.  A block-table entry outside [0, num_blocks) of a used page reads as a page of zeros.
 */
int amla_mla_decode_fp8_workspace_size(int B, int Sq, int H, int max_blocks_per_seq, int device, size_t* bytes_out);
int amla_mla_decode_fp8(const void* q, const void* kv_cache_e4m3, float kv_scale, const int32_t* block_table,
                        const int32_t* seqlens, float softmax_scale, int B, int Sq, int H, int num_blocks,
                        int max_blocks_per_seq, void* out, float* lse, void* workspace, size_t workspace_bytes,
                        void* cuda_stream, int flags);

/* Synchronises `cuda_stream` and reads the status word the kernels keep at the start of the
 * workspace: AMLA_OK, or AMLA_ERR_DEVICE_TIMEOUT if a bounded wait inside a kernel expired (the
 * kernel then returned early and the outputs are undefined).  Optional. */
int amla_check_status(const void* workspace, void* cuda_stream);

/*
 * Diagnostic: shows that a bounded device-side wait reports instead of hanging.  Launches a one-warp kernel that
 * waits, with the wait routine of the decode kernels and a limit of `limit_ns` nanoseconds (1 .. 100 000 000),
 * on a barrier nothing arrives on; when the limit passes it stores the time-out status in the first word of
 * `workspace` (device, 4-byte aligned, at least 4 bytes) and ends.  amla_check_status(workspace, stream) then
 * returns AMLA_ERR_DEVICE_TIMEOUT; the next decode call on that workspace resets the word.  No decode work runs.
 */
int amla_wait_selftest(void* workspace, unsigned long long limit_ns, void* cuda_stream);

/*
 * Debug aid, host only: checks HOST copies of the paging inputs before a decode call.  Every seqlens[b] must lie
 * in [0, 64 * max_blocks_per_seq] and every block_table entry that the sequence uses (the first
 * ceil(seqlens[b] / 64) of row b) in [0, num_blocks).  Returns AMLA_OK, or AMLA_ERR_INVALID_ARG with the
 * offending sequence in *bad_seq and entry index in *bad_block (-1 when the length itself is out of range);
 * either pointer may be NULL.  (The kernels never fault on a bad page index -- an out-of-range TMA coordinate
 * reads as zeros -- so such a mistake shows up as wrong results only; this check names it.)  Nothing is launched.
 */
int amla_validate_paging_host(const int32_t* block_table, const int32_t* seqlens, int B, int num_blocks,
                              int max_blocks_per_seq, int* bad_seq, int* bad_block);

/* Number of kernels the most recent amla_mla_decode[_ex] call on this thread launched. */
int amla_last_launch_count(void);

/* Measurement aid (the one piece of per-thread state in the library): when enabled, every decode call
 * on this thread records CUDA events on its stream around its launches: before the schedule kernel
 * (which only batches of more than 2048 items have; otherwise that interval is empty), between it and
 * the decode kernel, between decode and combine, and after.  The events are created on the first
 * enable and live until exit. */
int amla_profile_enable(int on);

/* Waits for the last profiled call on this thread and writes the elapsed milliseconds of the three
 * intervals (schedule, decode, combine) to ms3[0..2].  AMLA_ERR_INVALID_ARG if nothing was profiled. */
int amla_profile_last_ms(float* ms3);

/*
 * Host mirror of the device-side split-KV schedule (the plan is not in the paper; it exists because
 * B * ceil(Sq*H/128) work items are far fewer than the SMs).  For Sq*H <= 128 the items are (sequence, 128-row
 * block) pairs, their tiles 64-key pages, and every non-empty item but the first is preceded by 10 overhead
 * positions that stand for the cost of starting an item; for Sq*H > 128 the items are (sequence, 256-row block)
 * pairs, the tiles 128 keys (two pages) and the overhead 5 positions.  Items in order form one linear range
 * that is cut into num_parts equal parts.
 * For every (part, item) intersection ("unit") one record of 6 int32 is written:
 *   part, item, tile_begin, tile_end (within the item), slot (-1 = writes out/lse directly,
 *   otherwise index of its fp32 partial), n_split of the item.
 * seqlens is a HOST array here.  Returns the number of units, or a negative amla_status
 * (AMLA_ERR_WORKSPACE if max_units is too small).
 */
int amla_plan_host(const int32_t* seqlens, int B, int Sq, int H, int num_parts, int32_t* units,
                   int max_units);

#ifdef __cplusplus
}
#endif
#endif /* AMLA_H_ */
