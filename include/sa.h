/* sa.h — C ABI of the shift-accumulate decode-attention library for NVIDIA B200 (sm_100a).
 *
 * The library computes decode-time attention of one query vector per head against a key
 * cache stored as signed power-of-two fixed-point codes, after "Shift-Accumulate Attention:
 * Multiplier-Free Query-Key Products for Transformer Decoding".  Citations below name the
 * paper's sections and equations.
 *
 * General rules for every function
 *   - `extern "C"`, returns an sa_status, never throws, never aborts.
 *   - Pointers are DEVICE pointers unless the parameter name ends in `_host`.  All memory is
 *     owned by the caller; the library allocates no device memory and keeps no state between
 *     calls (the one exception, a fixed scratch array, is sa_decode_attention_static).
 *   - Work is enqueued on the caller's stream (`sa_stream` is a `cudaStream_t`); no function
 *     synchronises.  Arguments are validated on the host before anything is launched; a call
 *     that returns an error has launched nothing.
 *   - Half-precision data is passed as IEEE binary16 bit patterns in `uint16_t`.
 *   - Inputs must be finite.
 *   - Query head h reads KV head h / (n_q_heads / n_kv_heads).
 *
 * Number formats (section II-A, II-D, II-E)
 *   Key element  K^_jm = s_j * sigma * (1 + j/2^k) * 2^-e,  e in 0..6, code e = 7 is an exact
 *   zero, k in {0, 1, 2, 4} mantissa bits (PoT-4, PoT-M1, PoT-M2, PoT-M4), s_j = the key
 *   vector's largest magnitude (binary16).  Rounding is to the nearest codeword in log2 on the
 *   grid continued below e = 6; an element that rounds to e >= 7 becomes the zero code.
 *   Canonical code byte: bit 7 sign (1 = negative), bits 6..4 e, bits 3..0 the mantissa
 *   left-aligned (j << (4 - k)); zero is 0x70.
 *   Query  Q_im ~ Delta_i * qhat_im, qhat in [-127, 127], Delta_i = amax_i / 127.
 *   Value  V_jm ~ vhat_jm * 2^-g_j, vhat INT8, g_j the largest integer with amax_j * 2^g_j <= 127.
 *
 * Cache layout (this library's own; section II-F only fixes what is stored)
 *   The page pool is n_pages * n_kv_heads blocks of `page_bytes`; block (p, h) starts at
 *   ((size_t)p * n_kv_heads + h) * page_bytes and holds page_tokens = 64 tokens of KV head h as two
 *   halves of page_bytes / 2 bytes, tokens 0..31 and 32..63.  A half is what a decode kernel stages for
 *   one 32-key tile, with a single bulk copy; the offsets below are relative to the half, t = token % 32:
 *     kcode_off: key codes in 16-byte chunks, chunk c of token t at (c * 32 + t) * 16.
 *                Byte container (any k): chunk c holds elements 16c .. 16c+15, one byte each:
 *                sign << 7 | mantissa field << 3 | g, with the canonical byte's 4-bit mantissa
 *                field and g = 7 - e (g = 0 for the zero code), so that g - 1 is the shift amount,
 *                the mantissa field times 8 a table offset, and zeroed memory reads as zero codes.  Nibble container (PoT-4 only): chunk c holds
 *                elements 32c .. 32c+31, byte i = element 32c+2i in the low nibble and 32c+2i+1
 *                in the high nibble, nibble = sign << 3 | g.
 *     meta_off : 32 records of 4 bytes: binary16 s_j, int8 g_j, one zero byte.
 *     v_off    : vhat, int8, in 16-byte chunks like the keys: chunk c (dims 16c .. 16c+15) of token t
 *                at (c * 32 + t) * 16.
 *   For code = SA_KV_FP16 each half holds unquantised binary16 data: K and then V, each in
 *   16-byte chunks of 8 elements (chunk c of token t at (c * 32 + t) * 16), no metadata.
 */
#ifndef SA_H_
#define SA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct CUstream_st* sa_stream; /* a cudaStream_t; NULL is the default stream */

typedef enum {
    SA_OK = 0,
    SA_ERR_INVALID_ARG = 1, /* null pointer, non-positive size, inconsistent head counts ...   */
    SA_ERR_UNSUPPORTED = 2, /* head_dim, code, layout or head-room outside what is implemented */
    SA_ERR_ALIGNMENT = 3,   /* a pointer is not aligned as documented                          */
    SA_ERR_CAPACITY = 4,    /* workspace or staging buffer too small, page table too short     */
    SA_ERR_CUDA = 5         /* the CUDA runtime refused a launch or a copy                     */
} sa_status;

/* Key code family: the value is k, the number of mantissa bits (eq. (2), eq. (5)). */
enum { SA_POT4 = 0, SA_POTM1 = 1, SA_POTM2 = 2, SA_POTM4 = 4, SA_INT8 = 8, SA_KV_FP16 = 16 };
/* SA_INT8 is the comparison code of section III / VI (an INT8 multiply-accumulate kernel built on the
 * same skeleton as the shift kernels): uniform INT8 keys, khat = round(K * 127 / amax) with the row maximum as
 * scale, stored one byte per element in the byte container (132 bytes per key at d = 64, the same
 * as PoT-M4); scores are integer dot products evaluated with dp4a.  Everything else (query and
 * value quantisers, softmax, A.V, merge, cache layout) is shared with the power-of-two codes. */
/* How key codes are stored in a page.
 * SA_KLAYOUT_BYTE: one byte per element (any code).
 * SA_KLAYOUT_NIBBLE: SA_POT4 only, two 4-bit codes (sign, exponent) per byte.
 * SA_KLAYOUT_PLANAR: SA_POTM1 / SA_POTM2 only, the dense 5- and 6-bit form of section II-F (the
 *   paper's 109-byte PoT-M1 record): the sign/exponent nibbles as in SA_KLAYOUT_NIBBLE, followed at
 *   kcode_off + 32 * head_dim / 2 (within each half of the block) by k bit planes of the mantissa, plane b
 *   holding head_dim / 8 bytes per token (bit m % 8 of byte m / 8 = bit b of element m's mantissa), the
 *   half's 32 tokens after one another.  108 / 116 bytes per key at head_dim = 64 against 132 in the byte container. */
enum { SA_KLAYOUT_BYTE = 0, SA_KLAYOUT_NIBBLE = 1, SA_KLAYOUT_PLANAR = 2 };
/* flags */
#define SA_FLAG_HADAMARD 1u /* rotate Q and K by the normalised Walsh-Hadamard matrix before quantising */
/* Decode kernels only, mantissa codes (PoT-M1 / M2 / M4) only, off by default: execute the left shift of
 * eq. (3), (4) on the integer multiplier.  Each key element is decoded once, for the whole query group, to
 * sigma * 2^(F - k - e) (0 for the zero code) and every (query, element) update is one integer multiply-add
 * by that power of two instead of a shift followed by the sign multiply-add.  The INT32 scores are the same
 * bit for bit.  This uses the multiplier array as a barrel shifter, so it is not the paper's multiplier-free
 * datapath; it is the mid-point between the shift kernels and the INT8 multiply-accumulate comparison
 * (section III), and is reported as such.  (PoT-4 has no shift left in its key loop: SA_ERR_UNSUPPORTED.) */
#define SA_FLAG_SHIFT_BY_MULTIPLY 2u
/* Decode kernels only, power-of-two codes only, off by default: every sign flip and add of the integer score
 * (eq. (3)) is issued as logic and add instructions (exclusive-or with the sign mask, subtract, add) instead
 * of one multiply-add by +1 / -1, so that no instruction of the score datapath touches the multiplier array.
 * The INT32 scores are the same bit for bit.  It is the strictly multiplier-free form of the default kernels
 * and is slower than them on this GPU, whose shift/logic/add pipe is the busier one; it exists to be measured
 * beside the default, SA_FLAG_SHIFT_BY_MULTIPLY and the INT8 multiply-accumulate comparison.  Excludes
 * SA_FLAG_SHIFT_BY_MULTIPLY. */
#define SA_FLAG_ADD_ON_ALU 4u

typedef struct {
    int head_dim;    /* 64 or 128 */
    int n_q_heads;   /* multiple of n_kv_heads */
    int n_kv_heads;
    int code;        /* SA_POT4 / SA_POTM1 / SA_POTM2 / SA_POTM4, SA_INT8 (comparison), or SA_KV_FP16 (FP16 baseline cache) */
    int klayout;     /* SA_KLAYOUT_BYTE, SA_KLAYOUT_NIBBLE (only with SA_POT4) or SA_KLAYOUT_PLANAR (SA_POTM1 / SA_POTM2) */
    int headroom_F;  /* fixed-point head-room F of eq. (3); 0 selects the default E + k = 6 + k.
                        Must satisfy F >= 6 + k (eq. (4): every shift is a left shift) and
                        head_dim * 127 * (2^(k+1) - 1) * 2^(F - k) < 2^31 (INT32 accumulator) */
    int page_tokens; /* 64 */
    unsigned flags;  /* SA_FLAG_HADAMARD | SA_FLAG_SHIFT_BY_MULTIPLY | SA_FLAG_ADD_ON_ALU */
} sa_config;

typedef struct {
    size_t page_bytes; /* bytes of one (page, KV head) block */
    size_t kcode_off;  /* offsets inside each 32-token half of a block (the second half starts at page_bytes / 2) */
    size_t meta_off;
    size_t v_off;
    size_t align;      /* required alignment of the pool base pointer */
} sa_layout;

typedef struct {
    void* pages;               /* page pool, n_pages * n_kv_heads * page_bytes bytes                     */
    const int32_t* page_table; /* [batch, max_pages_per_seq]: pool index of each sequence's logical page */
    int32_t* seq_lens;         /* [batch]: tokens already cached per sequence                            */
    int batch;
    int max_pages_per_seq;
    int n_pages;
} sa_cache;

int sa_version(void);
const char* sa_status_string(sa_status s);

/* Byte layout of one (page, KV head) block for this configuration.  Host only, no CUDA call. */
sa_status sa_get_layout(const sa_config* cfg, sa_layout* out);

/* Bytes of scratch that sa_decode_attention / sa_decode_attention_fp16 need for a cache with
 * `batch` sequences of at most `max_pages_per_seq` pages (split-K partial results, section II-F:
 * the kernel grid has a split dimension; for batches of 2 to 128 sequences also two words per sequence,
 * in which the decode kernel tells the merge kernel how it dealt the grid's blocks to the sequences: in
 * proportion to their cached lengths, so that a batch of unequal lengths keeps the machine as full as one
 * of equal lengths).  Host only; the one CUDA call it may make reads the number of
 * multiprocessors of the CURRENT device (once per device), because the split count is planned for it: ask on
 * the device the decode calls will run on (without a device the figure of a B200 is used).  The scratch needs
 * no initialisation and may be shared by calls that do not overlap on the GPU. */
sa_status sa_workspace_bytes(const sa_config* cfg, int batch, int max_pages_per_seq, size_t* out);

/* Key encode (eq. (2), eq. (5); nearest-in-log2 rounding, section II-D).
 * K [n, n_kv_heads, head_dim] binary16 -> codes [n, n_kv_heads, head_dim] canonical bytes and
 * scales [n, n_kv_heads] binary16.  With SA_FLAG_HADAMARD each head vector is rotated first. */
sa_status sa_encode_keys(const sa_config* cfg, const uint16_t* K, int64_t n, uint8_t* codes,
                         uint16_t* scales, sa_stream stream);

/* Query quantisation (eq. (2)): Q [batch, n_q_heads, head_dim] binary16 -> q_hat int8 of the same
 * shape and delta [batch, n_q_heads] float.  With SA_FLAG_HADAMARD each head vector is rotated first. */
sa_status sa_quantise_query(const sa_config* cfg, const uint16_t* Q, int batch, int8_t* q_hat,
                            float* delta, sa_stream stream);

/* Value quantisation (section II-E: INT8 with a power-of-two per-token scale).
 * V [n, n_kv_heads, head_dim] binary16 -> v_hat int8 of the same shape and g [n, n_kv_heads] int8. */
sa_status sa_quantise_values(const sa_config* cfg, const uint16_t* V, int64_t n, int8_t* v_hat,
                             int8_t* g, sa_stream stream);

/* Append one token per sequence (the cache write of section II-F: the cache stores only
 * quantised data).  K_new, V_new [batch, n_kv_heads, head_dim] binary16.  Sequence b's token
 * is encoded / quantised as above and written at position seq_lens[b] of its page
 * page_table[b][seq_lens[b] / 64]; the page must already be mapped.  If bump_lens is non-zero
 * the kernel then increments seq_lens[b]; otherwise the caller does.  With code = SA_KV_FP16 the
 * binary16 data is stored as is. */
sa_status sa_append_kv(const sa_config* cfg, const sa_cache* cache, const uint16_t* K_new,
                       const uint16_t* V_new, int bump_lens, sa_stream stream);

/* Bulk build of a cache: K, V [sum_b T_b, n_kv_heads, head_dim] binary16, sequence b occupying
 * rows cu_lens_host[b] .. cu_lens_host[b+1] (HOST array of batch + 1 entries).  Writes tokens
 * 0 .. T_b - 1 of every sequence; does not touch seq_lens. */
sa_status sa_fill_kv(const sa_config* cfg, const sa_cache* cache, const uint16_t* K,
                     const uint16_t* V, const int64_t* cu_lens_host, sa_stream stream);

/* Decode attention over the quantised cache — the hot path (section II-B eq. (3), II-C eq. (4),
 * II-D eq. (5), II-E, II-F):
 *   Q is quantised (and rotated, if flagged) inside the kernel; for every cached key the integer
 *   score A = sum_m sigma * qhat * (2^k + j) << (F - k - e) is formed exactly in INT32 with
 *   shifts, sign flips and adds; logits z = A * Delta * s * 2^-F * log2(e) / sqrt(d) feed an
 *   online softmax whose running maximum is an integer in the log2 domain, so that every
 *   rescale is an exact power of two; O accumulates p * vhat * 2^-g (the paper's floating-point
 *   A.V); the key axis is split over thread blocks and the partial (M, l, O) triples are merged
 *   with exact power-of-two factors.
 *   The A.V products run on the tensor cores as tf32 x tf32 with FP32 accumulation (mma.m16n8k8): the INT8
 *   values are exact in tf32, and every weight p * 2^-g enters as the sum of two tf32 terms (its leading
 *   11 significant bits, and the remainder cut to 11 bits), so that a weight keeps about 21 significant
 *   bits: the relative error of one product is below 2^-21, against 2^-24 for an FP32 multiply; measured
 *   max |dO| against the CPU oracle is 2e-8 .. 6e-7.  The integer scores never touch the tensor cores.
 * Q [batch, n_q_heads, head_dim] binary16; O [batch, n_q_heads, head_dim] float.
 * A sequence with seq_lens[b] == 0 yields zeros.
 * dbg_scores (nullable): int32 [batch, n_q_heads, max_pages_per_seq * 64]; receives A for every
 * cached key (test hook; slows the call down).
 * Results are deterministic run to run (fixed split assignment, no floating-point atomics).
 * The kernels are launched with programmatic stream serialisation; the decode kernel reads Q
 * (and nothing else) before it waits for the preceding kernel in the stream, so Q must not be
 * written by a kernel that signals programmatic launch completion before it has written Q
 * (ordinary launches, copies and every kernel of this library satisfy that).  The split-K merge that ends
 * the call may release its dependents before it has written O: a following kernel that the CALLER launches
 * with the programmatic-serialisation attribute must execute its own grid-dependency wait before it reads O
 * or seq_lens (as that attribute always requires); ordinary launches and copies are ordered as usual. */
sa_status sa_decode_attention(const sa_config* cfg, const sa_cache* cache, const uint16_t* Q,
                              float* O, void* workspace, size_t workspace_bytes,
                              int32_t* dbg_scores, sa_stream stream);

/* The same decode step over an unquantised binary16 cache (cfg->code = SA_KV_FP16): textbook
 * softmax(Q K^T / sqrt(d)) V of eq. (1) with FP32 accumulation.  Baseline for a like-for-like
 * throughput ratio (the paper compared with a framework's FP16 attention). */
sa_status sa_decode_attention_fp16(const sa_config* cfg, const sa_cache* cache, const uint16_t* Q,
                                   float* O, void* workspace, size_t workspace_bytes,
                                   sa_stream stream);

/* One decode step of a layer in a single pass (section II-F: the cache stores only quantised data,
 * and the step both extends it and attends over it): equivalent to
 *   sa_append_kv(cfg, cache, K_new, V_new, 1, stream); sa_decode_attention(cfg, cache, Q, O, ...);
 * The warp of the decode kernel that owns the new token's 32-key tile encodes and writes the token
 * before it stages that tile, so the separate append kernel and its launch disappear from the
 * step; seq_lens[b] is incremented by the split-K merge kernel, after every block has read it.
 * As with sa_append_kv the token's page must already be mapped; if it is not, the token is not
 * written, the length stays, and the step attends over the old cache.
 * With more than 8 query heads per KV head the call runs the two kernels separately.  A binary16
 * cache (SA_KV_FP16) is served the same way by the binary16 decode kernel.  Same buffers,
 * alignment and workspace as sa_decode_attention; K_new, V_new [batch, n_kv_heads, head_dim]
 * binary16, 16-byte aligned. */
sa_status sa_decode_step(const sa_config* cfg, const sa_cache* cache, const uint16_t* Q,
                         const uint16_t* K_new, const uint16_t* V_new, float* O, void* workspace,
                         size_t workspace_bytes, sa_stream stream);

/* The paper's non-default option: attention weights quantised to powers of two and the
 * shift-based A.V (section II-E eq. (6), (7); section V-G), which makes the second product
 * multiplier-free too:
 *   M = ceil(max_j z_j), k_j = M - round(z_j) >= 0, weight 2^-k_j;
 *   O = 2^(-N - g_ref) * sum_{j: k_j <= k_max} vhat_j << (N - k_j + g_ref - g_j), divided by the
 *   sum of the kept weights; g_ref = min_j g_j.
 * M and g_ref are those of the whole sequence: the call runs the decode kernel's score phase
 * (rounded logits to the workspace), a second kernel with a per-tile INT32 accumulator, and the
 * split-K merge.  A key with k_j > k_max is dropped from numerator and normaliser, one whose
 * shift index is negative from the numerator only.  The paper prints no values for N (n_bits)
 * and k_max: 1 <= n_bits <= 18 (INT32 accumulator over a 32-key tile), 0 <= k_max <= n_bits.
 * Codes: SA_POT4 .. SA_POTM4 (not SA_INT8, not SA_KV_FP16).
 * workspace: at least sa_shiftav_workspace_bytes, 256-byte aligned, no initialisation needed.
 * dbg_scores (nullable) as in sa_decode_attention; dbg_rounded (nullable): int32 [batch, n_q_heads,
 * max_pages_per_seq * 64], receives round(z_j) for every cached key (test hook). */
sa_status sa_shiftav_workspace_bytes(const sa_config* cfg, int batch, int max_pages_per_seq, size_t* bytes);
sa_status sa_decode_attention_shiftav(const sa_config* cfg, const sa_cache* cache, const uint16_t* Q,
                                      float* O, void* workspace, size_t workspace_bytes, int n_bits,
                                      int k_max, int32_t* dbg_scores, int32_t* dbg_rounded,
                                      sa_stream stream);

/* The two decode entry points with their kernels selectable, for callers that want to time or
 * overlap them separately: stages is a bit mask, 1 = the main kernel (scores, softmax, A.V; writes
 * the split-K partials into the workspace), 2 = the merge of the partials into O.  stages = 3 is
 * what sa_decode_attention / sa_decode_attention_fp16 do.  (Measurement hook; the paper's
 * kernel description in section II-F has no counterpart of the split.) */
sa_status sa_decode_attention_stages(const sa_config* cfg, const sa_cache* cache, const uint16_t* Q,
                                     float* O, void* workspace, size_t workspace_bytes,
                                     int32_t* dbg_scores, int stages, sa_stream stream);
sa_status sa_decode_attention_fp16_stages(const sa_config* cfg, const sa_cache* cache,
                                          const uint16_t* Q, float* O, void* workspace,
                                          size_t workspace_bytes, int stages, sa_stream stream);

/* sa_decode_attention for callers that cannot allocate device memory.  (The paper has no
 * counterpart: this is a packaging variant of the same kernels, not a step of the method.)
 *
 * Who needs it: code that must call the decode step from a place where cudaMalloc (or a framework
 * allocator built on it) is off limits — a plug-in invoked inside another runtime's execution
 * callback, a serving loop whose device memory pool is frozen once start-up is over, a process
 * whose allocator may not be re-entered — and that therefore cannot produce the workspace the
 * normal entry point asks for.  Here the split-K partial results go into a fixed array compiled
 * into the library instead (SA_STATIC_SCRATCH_BYTES, 256-byte aligned).  The caller still passes
 * the cache, Q, O and, optionally, dbg_scores, exactly as for sa_decode_attention; results are
 * identical to it.  The call allocates nothing and frees nothing.
 *
 * Costs and rules:
 *   - Every GPU on which the library is used holds SA_STATIC_SCRATCH_BYTES from the moment the
 *     library's code is loaded on it until the process exits, whether or not this entry point is
 *     ever called.
 *   - The scratch bounds the problem: with S the split count the library picks for the cache
 *     shape, S * batch * n_q_heads * (head_dim + 2) * 4 bytes (plus 8 bytes per sequence for batches of
 *     2 to 128 sequences: exactly sa_workspace_bytes()) must fit.  A larger problem is
 *     refused with SA_ERR_CAPACITY and nothing is launched; use sa_decode_attention with a
 *     workspace of sa_workspace_bytes() for it.  (Batch 1, 32 query heads, head_dim 64 at any
 *     length fits; so does the ragged batch-16 configuration.)
 *   - The first call on each device looks up the array's device address (one CUDA runtime query,
 *     made with that device current, then cached).  Make that first call outside any stream
 *     capture; later calls on the same device do no such query.
 *   - All calls on a device share the one array, and it keeps whatever the previous call left.
 *     Nothing in it has to be cleared — each call overwrites every entry it later reads — but two
 *     calls that overlap on the GPU (different streams, or graphs replayed concurrently) race on
 *     it and corrupt each other's output.  Serialise them, or give the overlapping ones their own
 *     workspace through sa_decode_attention.
 *   - cfg->code must be one of the quantised key codes (the power-of-two codes or SA_INT8), not SA_KV_FP16. */
#define SA_STATIC_SCRATCH_BYTES (4u << 20)
sa_status sa_decode_attention_static(const sa_config* cfg, const sa_cache* cache, const uint16_t* Q,
                                     float* O, int32_t* dbg_scores, sa_stream stream);

/* Test hook for the failure path of the staged copies (the paper has no counterpart).  sa_decode_attention
 * in which the bulk copy of ONE tile — 32-token tile `tile` of sequence `b`, KV head `kv_head` — is never
 * issued and every wait for a copy gives up after 2^10 polls instead of 2^18.  The warp that owns that tile
 * finds its wait exhausted, abandons its remaining tiles and marks its block's partial result; the split-K
 * merge carries the mark into O: the rows of the query heads of `kv_head` in sequence `b` come out as NaN,
 * every other row is the ordinary result, and the call returns like any other (nothing is left in flight,
 * nothing waits without a bound).  Only head_dim 64, SA_POTM4 in the byte container, 8 query heads per KV
 * head, no flags: anything else is SA_ERR_UNSUPPORTED. */
sa_status sa_debug_decode_lost_copy(const sa_config* cfg, const sa_cache* cache, const uint16_t* Q, float* O,
                                    void* workspace, size_t workspace_bytes, int b, int kv_head, int tile,
                                    sa_stream stream);

/* Instruction-throughput micro-benchmark (measurement aid; the paper has no counterpart — it stands
 * in for the paper's disassembly-based operation counts, section III and Table V).  Launches `blocks`
 * blocks of 256 threads in which every thread runs iters * 64 instructions of one kind on 8
 * independent chains.  kind: 0 variable shift, 1 three-input logic op, 2 three-input add,
 * 3 multiply-add by one (an add issued on the FMA pipe), 4 byte permute, 5 shift/multiply-add mix,
 * 6 logic/multiply-add mix, 7 FP32 FMA, 8 packed FP32x2 FMA, 9 integer multiply-add, 10 dp4a,
 * 11 population count + add, 12 int8-to-float + add, 13 shift/logic/multiply-add mix, 14 / 15 the scalar video
 * shift-and-add (vshl ... wrap.add / clamp.add, the paper's Table V rows), 16 shift then add as two instructions,
 * 17 128-bit shared-memory load with every lane at one address, 18 / 25 64-bit shared-memory loads whose lanes
 * pick entries of one 128-byte row (regularly / irregularly), 19 int32-to-float, 20 float-to-int32 rounding up,
 * 21 ex2.approx, 22 byte-to-float, 23 the same as byte permute + FP32 add, 24 mul.hi.
 * `sink` is one device word (practically never written).  The caller times the launch. */
sa_status sa_pipe_microbench(int kind, int iters, int blocks, uint32_t* sink, sa_stream stream);

/* Test hook: unpack sequence b of a quantised cache into canonical arrays for its first
 * n_tokens tokens: codes [n_tokens, n_kv_heads, head_dim] canonical bytes, scales
 * [n_tokens, n_kv_heads] binary16, v_hat [n_tokens, n_kv_heads, head_dim] int8, g
 * [n_tokens, n_kv_heads] int8.  Any output pointer may be NULL.  n_tokens is given by the
 * caller (HOST value) and must not exceed max_pages_per_seq * 64. */
sa_status sa_debug_unpack(const sa_config* cfg, const sa_cache* cache, int b, int n_tokens,
                          uint8_t* codes, uint16_t* scales, int8_t* v_hat, int8_t* g,
                          sa_stream stream);

/* One decode step driven from HOST buffers (convenience for callers whose activations live on
 * the host): copies Q_host [batch, n_q_heads, head_dim], K_new_host and V_new_host
 * [batch, n_kv_heads, head_dim] (binary16, ideally pinned) into `staging`, appends the new token
 * to every sequence (incrementing seq_lens), runs the decode attention matching cfg->code
 * (quantised or SA_KV_FP16) and copies O [batch, n_q_heads, head_dim] float to O_host.
 * Everything is asynchronous on `stream`; synchronise it before reading O_host.
 * If all four host buffers are pinned and device-addressable (cudaHostAlloc / cudaHostRegister
 * memory under unified addressing), no copy engine is used: a small kernel fetches the inputs
 * and the merge kernel stores O directly into host memory.  That kernel reads the three input buffers
 * without waiting for kernels enqueued earlier on `stream` (they are host inputs): their contents must
 * be in place when the call is enqueued (or the graph holding it is launched), written by the host or by
 * work that has completed, not produced by a kernel still pending on the same stream.  Otherwise the buffers are copied
 * with cudaMemcpyAsync (a single copy for the inputs if Q_host, K_new_host and V_new_host follow
 * one another in one host buffer and their sizes are multiples of 256 bytes).
 * `staging` is device scratch of at least sa_staging_bytes(); not shared between overlapping calls. */
sa_status sa_staging_bytes(const sa_config* cfg, int batch, size_t* out);
sa_status sa_decode_step_host(const sa_config* cfg, const sa_cache* cache, const uint16_t* Q_host,
                              const uint16_t* K_new_host, const uint16_t* V_new_host, float* O_host,
                              void* staging, size_t staging_bytes, void* workspace,
                              size_t workspace_bytes, sa_stream stream);

#ifdef __cplusplus
}
#endif
#endif /* SA_H_ */
