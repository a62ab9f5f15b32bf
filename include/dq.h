/*
 * dq.h -- C ABI of the D-Quant hot path for NVIDIA B200 (sm_100a).
 *
 * D-Quant ("D-Quant: Driftable Entropy Coding for KV Cache Quantization") stores the
 * keys and values of every token in fixed-size, rANS-coded containers and decodes
 * them inside the decode-step attention kernel.  This library holds that path:
 *
 *   dq_build_tables           normal-derived rANS tables                  (Sec. 3.1, 4.2, 4.4)
 *   dq_encode_tokens          K/V bf16 -> containers + window means       (Fig. 1, Algorithm 1)
 *   dq_encode_tokens_rope     the same for keys handed over before their rotary embedding
 *   dq_decode_attention       q, containers -> attention output           (Algorithm 2, App. A)
 *   dq_decode_step            newest token encoded + attention, one overlapped launch sequence
 *   dq_decode_attention_residual / dq_window_append
 *                             the BF16 window of the most recent tokens   (Sec. 5.1)
 *   dq_decode_attention_multi several query tokens per sequence in one pass over the cache
 *   dq_decode_attention_static  dq_decode_attention without any allocation at call time
 *   dq_decode_tokens          containers -> symbols / dequantised values  (Algorithm 2; checks)
 *   dq_bf16_decode_attention  plain bf16-cache decode attention (comparison baseline)
 *
 * Conventions
 *   - A *stream* is the 128 values of one (token, KV head).  Its *record* is
 *     rec_bytes = floor(bits_per_elem * 128 / 8) bytes:
 *       [0:2) s fp16 LE | [2:4) o fp16 LE | [4:8) final rANS state u32 LE |
 *       [8:8+k) renormalisation bytes in decode order | zero padding.
 *     The container of Eq. (budget) is C = rec_bytes - 4 bytes, sigma = 32,
 *     B = 8C - 32 bits; rANS precision p = 8, state in [2^23, 2^31), byte-wise
 *     renormalisation.
 *   - Containers live in pages of 16 tokens: uint8 [num_pages][Hkv][16][rec_bytes].
 *     slot = page * 16 + index-in-page.  A record's address follows from (slot, head)
 *     alone (fixed stride, Sec. 4.1).
 *   - Token-wide streams (Sec. 5.1 "Implementation details": each token is quantised as a
 *     single group; 331 / 231-byte containers, 8 / 6 levels): tables built with
 *     heads_per_stream = hs > 1 describe streams of hs * 128 values, the hs consecutive KV
 *     heads of a token, each head rotated (and, for keys, centred on its window mean) on its
 *     own, with one (s, o) pair, one rANS state and one record per stream.  Their records
 *     (same field order, rec_bytes = floor(bits_per_elem * hs * 128 / 8)) are stored
 *     word-interleaved per page so that the 16 tokens of a page advance through memory
 *     together: uint8 [num_pages][Hkv / hs][rec_words][16][4], rec_words = ceil(rec_bytes / 4);
 *     byte i of the record of (page, group, token-in-page t) sits at
 *     ((page * (Hkv / hs) + group) * rec_words + i / 4) * 64 + t * 4 + i % 4; bytes past
 *     rec_bytes in the last word are zero.  The attention kernel addresses such an array in
 *     16-byte units with 32 bits: one token-wide container array may span at most 64 GiB
 *     (every page id in the page table times the page's bytes must stay below 2^36).
 *   - Key channel means: one per (sequence, window of 128 positions, KV head):
 *     int8 [S][max_windows][Hkv][128] and float scale [S][max_windows][Hkv];
 *     mean_j = scale * q_j, in the Hadamard-rotated domain.
 *   - Every pointer named "device" must be device memory reachable from the current
 *     device; the caller owns all of it, and the CUDA stream.  The library owns only
 *     dq_tables (host memory).  Calls validate their arguments, enqueue kernels on the
 *     given stream and return; 0 means "validated and enqueued".
 *   - Errors are returned, never thrown; nothing is launched when validation fails;
 *     no kernel traps or spins.
 *   - Codec variants (opt-in per table, dq_table_opts; the defaults are the paper's codec):
 *     * drift_early_exit: Algorithm 1's Drift bisects log2(lambda) in 12 steps; when every test
 *       passes it ends at a multiplier known beforehand.  The variant evaluates that multiplier
 *       first and returns its assignment when it meets the budget, otherwise runs the bisection
 *       (App. C: most streams have budget to spare).  Same record format.
 *     * sigma_bits = 24: records are [s fp16][o fp16][final state, 3 bytes LE][bytes ...]; the state
 *       lives in [2^15, 2^23) and B = 8C - 24 (Eq. budget), one more byte for symbols.  Key and
 *       value tables of one cache must agree on sigma_bits.  Per token-head streams only.
 *     * pair_symbols: one rANS symbol is the pair of levels of two consecutive values (2i, 2i + 1),
 *       u = m_2i M + m_2i+1, over the alphabet of M^2 pairs (Sec. 3.1: Eq. rans unchanged on a larger
 *       alphabet; the pair model is the product of the sharpened level model with itself, made
 *       integer by the same rule).  Algorithm 2 then takes 64 steps for 128 values, which is what
 *       halves the decode cost of the attention kernel; Algorithm 1's Drift assigns a pair at a
 *       time (argmin over the M^2 pairs of D_a + D_b + lambda r_ab, lowest u among equals; bracket
 *       16 (max D - min D)).  Same record layout and sizes.  At most 9 levels; key and value tables
 *       of one cache must agree.
 */
#ifndef DQ_H_
#define DQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define DQ_OK 0
#define DQ_ERR_ARG (-1)          /* null / out-of-range argument                     */
#define DQ_ERR_INFEASIBLE (-2)   /* the all-central stream does not fit the container */
#define DQ_ERR_UNSUPPORTED (-3)  /* head_dim != 128, GQA group > 8, record too large  */
#define DQ_ERR_WORKSPACE (-4)    /* workspace smaller than dq_decode_workspace_bytes  */
#define DQ_ERR_CUDA (-5)         /* a CUDA runtime call failed (see dq_last_cuda_error) */

#define DQ_MAX_LEVELS 16
#define DQ_MAX_PAIR_LEVELS 9      /* paired-symbol variant: levels 0..8 (their fp16 codes fit one byte) */
#define DQ_MAX_PAIRS 81
#define DQ_HEAD_DIM 128
#define DQ_PAGE_TOKENS 16
#define DQ_WINDOW_TOKENS 128
#define DQ_MAX_REC_BYTES 160      /* per token-head records                            */
#define DQ_MAX_WIDE_REC_BYTES 1024 /* records of streams that span several heads        */
#define DQ_MAX_STREAM_HEADS 8     /* heads per stream (1024 values)                    */
#define DQ_MAX_GROUP 8           /* query heads per KV head                           */

#define DQ_MEAN_COMPUTE 0
#define DQ_MEAN_REUSE 1

#define DQ_ROPE_HALF 1           /* rotary pairs (j, j + 64): the "rotate half" convention */
#define DQ_ROPE_PAIRS 2          /* rotary pairs (2j, 2j + 1)                              */

typedef struct dq_tables dq_tables; /* opaque, immutable after build, host memory */

typedef struct {
    int head_dim;   /* must be 128 */
    double alpha;   /* sharpening exponent p' ~ p^alpha (Sec. 4.4; paper: 1.4).  >= 0: used as
                       given (0 = uniform table).  < 0: smallest of 1.4, 1.5, ..., 32.0 whose
                       table has entropy <= B/128 and passes the feasibility test. */
    int has_mean;   /* 1: streams had a window mean removed (keys); 0: values          */
    int rotate;     /* 1: the library applies the per-head Hadamard rotation (Sec. 4.2) */
    int heads_per_stream; /* 0 or 1: one stream per (token, KV head); hs in 2..8: one stream per
                       hs consecutive KV heads of a token (hs = Hkv: the paper's token-wide
                       default, Sec. 5.1).  The model's n is then hs * 128. */
    /* Opt-in codec variants (0 = the paper's codec; see "Codec variants" below) */
    int drift_early_exit; /* 1: Drift first evaluates the multiplier its bisection ends at when every
                       test passes and stops there if the budget is met (encoder only; records
                       are read by the same decoder) */
    int sigma_bits;  /* 0 or 32: 32-bit final state, state in [2^23, 2^31).  24: 24-bit final state,
                       state in [2^15, 2^23), B = 8C - 24; per token-head streams only */
    int pair_symbols; /* 1: rANS symbols are pairs of levels (levels <= 9) */
} dq_table_opts;

typedef struct {
    int levels, head_dim, rec_bytes, container_bytes, budget_bits, mstar, has_mean, rotate;
    double alpha;
    int32_t f[DQ_MAX_LEVELS];      /* frequencies, sum 256            */
    int32_t c[DQ_MAX_LEVELS + 1];  /* cumulative frequencies          */
    float r[DQ_MAX_LEVELS];        /* -log2(f/256), bits (Algorithm 1) */
    uint32_t R[DQ_MAX_LEVELS];     /* ceil(r * 65536)                  */
    uint32_t lut[256];             /* f << 24 | (fp16 bits of level) << 8 | (z - c) */
    int heads_per_stream;          /* >= 1                                           */
    int rec_words;                 /* ceil(rec_bytes / 4): words per record in the interleaved layout */
    int sigma_bits;                /* 32 or 24: bits of final rANS state in a record    */
    int drift_early_exit;          /* 0 / 1                                             */
    /* paired-symbol variant (pair_symbols = 1); pair index u = a * levels + b, a = the even value's level.
       `lut` then holds  code(b) << 24 | f_u << 16 | code(a) << 8 | (z - c_u),  code(m) = high byte of fp16(m) */
    int pair_symbols, ustar;       /* 0 / 1; most probable pair                          */
    int32_t pair_f[DQ_MAX_PAIRS];  /* pair frequencies, sum 256                          */
    uint32_t pair_R[DQ_MAX_PAIRS]; /* ceil(65536 * -log2(pair_f / 256))                  */
} dq_table_info;

/* Probability model and rANS tables of one tensor kind (Sec. 3.1 "Entropy Coding",
 * Sec. 4.2 last paragraph, Sec. 4.4 "Distribution sharpening").  The probability of level
 * m is the N(0,1) mass of its cell on an M-level grid spanning +-E[max of n normals], n the
 * stream length (128, or hs * 128); frequencies are integers summing to 256.  Host only; needs
 * no GPU.  Returns DQ_ERR_INFEASIBLE when n * R[mstar] > 65536 * B (paired symbols: when
 * (n / 2) * pair_R[ustar] > 65536 * B).  *out is set only on DQ_OK. */
int dq_build_tables(int levels, double bits_per_elem, const dq_table_opts *opts, dq_tables **out);
void dq_free_tables(dq_tables *t);
int dq_tables_info(const dq_tables *t, dq_table_info *out);

/* Encoder (Fig. 1; Algorithm 1; Sec. 4.5 "Encoding"): Hadamard rotation, windowed channel
 * mean removal (keys), min-max affine grid, drift, least-squares refit, fp16 metadata,
 * second drift, rANS.  One warp per stream.
 *   tk / tv          tables for keys / values; either may be NULL to skip that tensor
 *   k_bf16, v_bf16   device, bf16 [T][Hkv][128]; finite values (any magnitude, subnormals included);
 *                    a NaN or an infinity gives an unspecified (in-bounds) record
 *   seq_id, pos      device int32 [T]: sequence and position of each token
 *   slot             device int32 [T]: physical slot; distinct per token
 *   k_cont, v_cont   device, containers as laid out above; only the T records written
 *   k_mean_q/scale   device, mean arrays as laid out above (keys with has_mean only)
 *   mean_mode        DQ_MEAN_COMPUTE: every maximal run of consecutive call tokens with the
 *                    same (seq_id, pos / 128) defines that window's mean (the tokens of a
 *                    window must be contiguous and ascending in pos).  DQ_MEAN_REUSE: stored
 *                    means are used; a token with pos % 128 == 0 first copies the previous
 *                    window's mean into its own window (window 0: zero); at most one such
 *                    token per sequence per call.
 *   status           device uint32[4], nullable, accumulated (not cleared): [0] streams that
 *                    fell back to the all-central assignment, [1] constant streams,
 *                    [2] rejected refits, [3] max record bytes used (atomicMax).
 * With token-wide tables (heads_per_stream = hs > 1; both tables must agree, Hkv % hs == 0) one
 * CTA of hs warps encodes a stream and the containers use the interleaved layout.
 * Calls with many streams (prefill, bulk encodes) run batch kernels that code 32 streams per CTA;
 * the records are the same.  The option DQ_OPT_ENCODE_BATCH_MIN (a stream count, dq_set_option)
 * moves the size from which they are used.
 * Errors: DQ_ERR_ARG for null / negative arguments, DQ_ERR_UNSUPPORTED for mismatched
 * heads_per_stream, DQ_ERR_CUDA on launch failure. */
int dq_encode_tokens(const dq_tables *tk, const dq_tables *tv, const void *k_bf16,
                     const void *v_bf16, int T, int Hkv, const int32_t *seq_id,
                     const int32_t *pos, const int32_t *slot, uint8_t *k_cont, uint8_t *v_cont,
                     int8_t *k_mean_q, float *k_mean_scale, int max_windows, int mean_mode,
                     uint32_t *status, void *cuda_stream);

/* dq_encode_tokens for keys handed over before their rotary position embedding, so that the
 * embedded keys never exist in bf16 (the paper encodes post-RoPE keys, Sec. 5.1; it does not
 * describe this fusion): k_bf16 is rotated in binary32 by the angle tables of each token's
 * position, then goes through the same pipeline (Hadamard, window mean, grid, drift, rANS);
 * window means (DQ_MEAN_COMPUTE) are those of the embedded keys.  Values are untouched.
 *   rope_cos, rope_sin   device float [positions][64], 16-byte aligned, positions > every pos[t]:
 *                        cos / sin of position * frequency j (the caller owns the frequency rule)
 *   rope_style           DQ_ROPE_HALF or DQ_ROPE_PAIRS; 0 (with NULL tables) = dq_encode_tokens
 * Per pair (a, b): (a cos - b sin, b cos + a sin), every product and sum rounded once. */
int dq_encode_tokens_rope(const dq_tables *tk, const dq_tables *tv, const void *k_bf16,
                          const void *v_bf16, int T, int Hkv, const int32_t *seq_id,
                          const int32_t *pos, const int32_t *slot, uint8_t *k_cont, uint8_t *v_cont,
                          int8_t *k_mean_q, float *k_mean_scale, int max_windows, int mean_mode,
                          const float *rope_cos, const float *rope_sin, int rope_style,
                          uint32_t *status, void *cuda_stream);

/* Bytes of scratch dq_decode_attention needs (split-K partials and a work counter). */
size_t dq_decode_workspace_bytes(int B, int Hq, int max_pages);

/* Decode-step attention over the compressed cache (Sec. 4.5 "Decoding"; Algorithm 2;
 * Appendix A fold-key / fold-value): every record is rANS-decoded in shared memory, the
 * levels feed tensor-core contractions, the affine terms are applied after them, softmax
 * is online, token ranges are split over CTAs and merged by log-sum-exp.
 *   q_bf16      device bf16 [B][Hq][128]; the library rotates it when keys are rotated
 *   page_table  device int32 [B][max_pages]: physical page of tokens 16 i .. 16 i + 15
 *   seq_lens    device int32 [B]; 0 gives a zero output row; must be <= 16 * max_pages
 *   out_bf16    device bf16 [B][Hq][128] (nullable if out_f32 is given)
 *   out_f32     device float [B][Hq][128], nullable: the result before bf16 rounding
 *   workspace   device, >= dq_decode_workspace_bytes(B, Hq, max_pages), 16-byte aligned
 * Hq must be a multiple of Hkv with Hq / Hkv <= 8, and B <= 4096 (else DQ_ERR_UNSUPPORTED: the
 * kernels keep the per-sequence block prefix sums in shared memory). */
int dq_decode_attention(const dq_tables *tk, const dq_tables *tv, const void *q_bf16,
                        const uint8_t *k_cont, const uint8_t *v_cont, const int8_t *k_mean_q,
                        const float *k_mean_scale, int max_windows, const int32_t *page_table,
                        int max_pages, const int32_t *seq_lens, int B, int Hq, int Hkv,
                        float sm_scale, void *out_bf16, float *out_f32, void *workspace,
                        size_t workspace_bytes, void *cuda_stream);

/* Decode-step attention with a BF16 residual window (Sec. 5.1 "Implementation details": the
 * most recent 128 tokens are retained in BF16).  As dq_decode_attention, plus per sequence
 * resid_lens[b] <= resid_cap further tokens that follow the seq_lens[b] compressed ones and are
 * stored uncompressed and unrotated:
 *   resid_k_bf16, resid_v_bf16   device bf16 [B][resid_cap][Hkv][128]
 *   resid_lens                   device int32 [B]
 * They join the same softmax (logits sm_scale * q.k) and contribute a_t v_t to the output.  When
 * a window fills, the caller encodes its 128 tokens with dq_encode_tokens(DQ_MEAN_COMPUTE): the
 * window then gets its own channel mean.  All three pointers NULL = dq_decode_attention. */
int dq_decode_attention_residual(const dq_tables *tk, const dq_tables *tv, const void *q_bf16,
                                 const uint8_t *k_cont, const uint8_t *v_cont, const int8_t *k_mean_q,
                                 const float *k_mean_scale, int max_windows, const int32_t *page_table,
                                 int max_pages, const int32_t *seq_lens, const void *resid_k_bf16,
                                 const void *resid_v_bf16, const int32_t *resid_lens, int resid_cap, int B,
                                 int Hq, int Hkv, float sm_scale, void *out_bf16, float *out_f32,
                                 void *workspace, size_t workspace_bytes, void *cuda_stream);

/* One decode step of a layer in a single call: encode the newest token of every sequence
 * (dq_encode_tokens with DQ_MEAN_REUSE: token b is the token at position seq_lens[b] - 1 of
 * sequence b; sequences of length 0 have none) and attend over the whole cache including it
 * (dq_decode_attention).  Same results as those two calls; the point is the schedule: the
 * attention kernel starts while the encoder still runs, works through every block that does not
 * hold a newest token first (work items come from a global counter, so the few SMs that host the
 * encoder simply take fewer), and waits for the encoder only before the first block that does.
 * Per token-head streams only (heads_per_stream = 1: DQ_ERR_UNSUPPORTED otherwise).
 *   k_new_bf16, v_new_bf16   device bf16 [B][Hkv][128]
 *   slot_new                 device int32 [B]: physical slot of each newest token
 *   seq_lens                 device int32 [B]: lengths including the newest token
 *   status                   as in dq_encode_tokens (nullable)
 * Other arguments as in dq_decode_attention.  Not to be mixed on one stream with work that
 * reads `workspace` concurrently; the first 16 bytes of the workspace carry the hand-over state.
 * The attention CTAs take the hand-over on a flag they poll a bounded number of times (65 536 polls,
 * 64 ns apart; the option DQ_OPT_STEP_POLL_LIMIT, dq_set_option, replaces the count);
 * a CTA that gives up waits for the preceding kernels instead: same results, no overlap. */
int dq_decode_step(const dq_tables *tk, const dq_tables *tv, const void *k_new_bf16, const void *v_new_bf16,
                   const int32_t *slot_new, const void *q_bf16, uint8_t *k_cont, uint8_t *v_cont,
                   int8_t *k_mean_q, float *k_mean_scale, int max_windows, const int32_t *page_table,
                   int max_pages, const int32_t *seq_lens, int B, int Hq, int Hkv, float sm_scale,
                   void *out_bf16, float *out_f32, void *workspace, size_t workspace_bytes,
                   uint32_t *status, void *cuda_stream);

/* Appends one new token per sequence to the BF16 residual window and counts it (the serving
 * policy of Sec. 5.1: new tokens enter the window; when it holds resid_cap tokens the caller encodes
 * them with dq_encode_tokens(DQ_MEAN_COMPUTE) and resets resid_lens[b] to 0).
 *   k_bf16, v_bf16               device bf16 [B][Hkv][128], 16-byte aligned: the new tokens
 *   resid_k_bf16, resid_v_bf16   device bf16 [B][resid_cap][Hkv][128], 16-byte aligned
 *   resid_lens                   device int32 [B], read and incremented; a sequence whose window is
 *                                full (or whose count is negative) is left unchanged */
int dq_window_append(const void *k_bf16, const void *v_bf16, void *resid_k_bf16, void *resid_v_bf16,
                     int32_t *resid_lens, int resid_cap, int B, int Hkv, void *cuda_stream);

/* Attention for q_len query tokens per sequence in one pass over the cache (speculative
 * decoding, short chunks of prefill); the paper's kernel is the q_len = 1 case (Sec. 4.5).
 *   q_bf16, out_*   [B][q_len][Hq][128]
 *   seq_lens, resid_lens   count every token of the sequence including the q_len newest ones, whose
 *                   K/V the caller has already stored (compressed, or in the BF16 window).  Query token
 *                   i (0 = oldest) sees the first seq_lens[b] + resid_lens[b] - (q_len - 1 - i) tokens of
 *                   the sequence: all compressed tokens come before all window tokens.
 *   workspace       >= dq_decode_workspace_bytes(B, Hq * min(q_len, 8 / (Hq / Hkv)), max_pages)
 * Up to 8 (query token, head) rows of a KV head share one decode of its streams: while
 * q_len * (Hq / Hkv) <= 8 the cost is that of q_len = 1; more query tokens are handled in
 * ceil(q_len / (8 / (Hq / Hkv))) passes over the cache inside this call.
 * resid_* may be NULL (no window). */
int dq_decode_attention_multi(const dq_tables *tk, const dq_tables *tv, const void *q_bf16, int q_len,
                              const uint8_t *k_cont, const uint8_t *v_cont, const int8_t *k_mean_q,
                              const float *k_mean_scale, int max_windows, const int32_t *page_table,
                              int max_pages, const int32_t *seq_lens, const void *resid_k_bf16,
                              const void *resid_v_bf16, const int32_t *resid_lens, int resid_cap, int B,
                              int Hq, int Hkv, float sm_scale, void *out_bf16, float *out_f32,
                              void *workspace, size_t workspace_bytes, void *cuda_stream);

/* dq_decode_attention for callers that must not allocate (the paper has no counterpart: this
 * is a packaging variant of the same kernels, not part of the method).
 *
 * Some callers cannot obtain the workspace dq_decode_attention asks for: an engine whose device
 * memory is handed out once at start-up and frozen, a plug-in running under a host program that
 * owns every allocation, a real-time loop where an allocator call (which may synchronise the
 * device or fail when memory is fragmented) is not acceptable.  For them the library carries its
 * own scratch: a fixed array of DQ_STATIC_SCRATCH_BYTES in device global memory that every GPU
 * loading the library holds until the process (context) ends.  This entry point passes that
 * array to the kernels in place of a workspace and makes no cudaMalloc / cudaFree call and no
 * call into any allocating library; inputs and outputs are still the caller's.
 *
 *   - Arguments, layouts and results are those of dq_decode_attention, minus the workspace.
 *   - Limit: dq_decode_workspace_bytes(B, Hq, max_pages) must not exceed
 *     DQ_STATIC_SCRATCH_BYTES; larger calls return DQ_ERR_WORKSPACE before anything is
 *     launched and dq_last_cuda_error() then says how many bytes were needed.
 *   - The first call on each device looks up the array's device address (current device must
 *     be the one the call is meant for); make that first call outside any stream capture.
 *   - All calls share the one array, which keeps whatever the previous call left in it; the
 *     kernels reset what they need (work counter, prefix sums) themselves.  Two calls that
 *     overlap on the GPU (different streams, or different host threads) race on it: serialise
 *     them.  dq_profile_enable has no effect on this entry point. */
#define DQ_STATIC_SCRATCH_BYTES (4u << 20)
int dq_decode_attention_static(const dq_tables *tk, const dq_tables *tv, const void *q_bf16,
                               const uint8_t *k_cont, const uint8_t *v_cont, const int8_t *k_mean_q,
                               const float *k_mean_scale, int max_windows, const int32_t *page_table,
                               int max_pages, const int32_t *seq_lens, int B, int Hq, int Hkv,
                               float sm_scale, void *out_bf16, float *out_f32, void *cuda_stream);

/* Check/debug export of Algorithm 2: decode T * Hkv records to symbols and to dequantised
 * values in the rotated domain, xhat = fma(m, s, o) (+ mean for keys).
 *   symbols  device uint8 [T][Hkv][128], nullable;  dequant  device float, same shape, nullable
 *   mean arrays may be NULL when t has no mean. */
int dq_decode_tokens(const dq_tables *t, const uint8_t *cont, const int8_t *mean_q,
                     const float *mean_scale, int max_windows, const int32_t *seq_id,
                     const int32_t *pos, const int32_t *slot, int T, int Hkv, uint8_t *symbols,
                     float *dequant, void *cuda_stream);

/* Comparison baseline (no counterpart in the paper's method: its reference point is bf16
 * FlashAttention-2, Sec. 5.1): split-K decode attention over an un-quantised bf16 cache
 * laid out [num_pages][Hkv][16][128].  Same page table, workspace and outputs as above. */
int dq_bf16_decode_attention(const void *q_bf16, const void *k_bf16_pages, const void *v_bf16_pages,
                             const int32_t *page_table, int max_pages, const int32_t *seq_lens,
                             int B, int Hq, int Hkv, float sm_scale, void *out_bf16,
                             void *workspace, size_t workspace_bytes, void *cuda_stream);

/* Process-wide tuning options (no counterpart in the paper).  value < 0 restores the default.
 *   DQ_OPT_STEP_POLL_LIMIT    dq_decode_step: polls of the hand-over flag before an attention CTA
 *                             falls back to waiting for the preceding kernels (0: at once;
 *                             at most 2^24).  Same results either way.
 *   DQ_OPT_ENCODE_BATCH_MIN   encoder: number of streams in a call from which the batch kernels
 *                             are used (0: always).  Same records either way.
 * Returns DQ_ERR_ARG for an unknown key or an out-of-range value.  dq_get_option returns the value
 * set (-1: default in force, or unknown key). */
#define DQ_OPT_STEP_POLL_LIMIT 1
#define DQ_OPT_ENCODE_BATCH_MIN 2
int dq_set_option(int key, long long value);
long long dq_get_option(int key);

/* Measurement aid (no counterpart in the paper): while enabled (on > 0), every on-th
 * dq_decode_attention call records CUDA events on its stream around the fused kernel (up to
 * 4096 records; the events keep that call's kernels from overlapping their neighbours).
 * dq_profile_read waits for them, writes the kernel durations in milliseconds (host array,
 * call order) and clears the record; returns how many it wrote.  Not thread-safe. */
void dq_profile_enable(int on);
int dq_profile_read(float *ms_out, int max_records);

/* Measurement aid (no counterpart in the paper): the bare symbol step of Algorithm 2 as the fused
 * kernel executes it, on byte streams held in shared memory -- no tiles, contractions, softmax or
 * global traffic.  `ctas` CTAs of `threads` threads (a multiple of 32, <= 1024) each make `reps`
 * passes of 128 symbols per chain with `chains` (1 or 2) independent chains per lane; the caller
 * times the launch with events on its stream.  Symbols decoded = ctas * threads * chains * 128 * reps.
 *   t       any per token-head table (its 256-entry table is the one looked up)
 *   bytes   device, nbytes >= 4096 arbitrary bytes the streams are filled from
 *   out     device uint32 [ctas * threads]: a checksum per thread (keeps the loop alive) */
int dq_microbench_decode_loop(const dq_tables *t, const uint8_t *bytes, size_t nbytes, int ctas,
                              int threads, int chains, int reps, uint32_t *out, void *cuda_stream);

const char *dq_strerror(int code);
/* Text of the last CUDA error seen by this thread's calls ("" if none). */
const char *dq_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* DQ_H_ */
