// Internal declarations shared by the library's translation units (not part of the ABI).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "dq.h"

// Table of one tensor kind as the kernels see it; passed by value as a kernel parameter
// (constant bank), so building tables needs no device memory.
struct DqDevTable {
    int M, rec, mstar, budget_bits;
    int has_mean, rotate;
    int hs, rec_words;           // heads per stream (>= 1); words per record (interleaved layout, hs > 1)
    int sigma, early_exit;       // bits of final state in a record (32 / 24); Drift tries its end multiplier first
    int pair, ustar;             // paired-symbol variant: rANS symbols are pairs u = a M + b; most probable pair
    uint32_t enc_rcp[DQ_MAX_LEVELS];  // encoder, Eq. rans Enc by reciprocal: floor(x / f) = umulhi(x, rcp) >> rsh
    uint32_t enc_aux[DQ_MAX_LEVELS];  // bias | (256 - f) << 10 | rsh << 19, bias = c (+ 255 when f = 1)
    float r[DQ_MAX_LEVELS];      // ideal cost in bits     (Algorithm 1)
    uint32_t R[DQ_MAX_LEVELS];   // ceil(r * 65536)
    uint32_t lut[256];           // f << 24 | fp16(level) << 8 | (z - c)   (Algorithm 2)
                                 // pair: code(b) << 24 | f << 16 | code(a) << 8 | (z - c), code = high byte of fp16(level)
};

// Encoder-side tables of the pair alphabet (paired-symbol variant); same packing as DqDevTable's.
struct DqPairEnc {
    uint32_t enc_rcp[DQ_MAX_PAIRS];
    uint32_t enc_aux[DQ_MAX_PAIRS];
    float r[DQ_MAX_PAIRS];
    uint32_t R[DQ_MAX_PAIRS];
};

struct dq_tables {
    dq_table_info info;
    DqDevTable dev;
    DqPairEnc penc;              // zero unless dev.pair
};

// dq_api.cu: process-wide options (dq_set_option); `dflt` is returned while an option is unset
int dq_opt_step_poll_limit(int dflt);
long long dq_opt_encode_batch_min(long long dflt);

// dq_tables.cu
int dq_host_build(int levels, double bits_per_elem, const dq_table_opts* opts, dq_tables* out);

// kernels' host launchers (each returns a cudaError_t from the launch)
cudaError_t dq_launch_means(const DqDevTable& tk, const void* k_bf16, int T, int Hkv,
                            const int32_t* seq_id, const int32_t* pos, int8_t* mean_q,
                            float* mean_scale, int max_windows, int mode, const float* rope_cos,
                            const float* rope_sin, int rope_style, cudaStream_t st);
struct DqEncodeArgs {
    const void* k_bf16;
    const void* v_bf16;
    const int32_t* seq_id;
    const int32_t* pos;
    const int32_t* slot;
    uint8_t* k_cont;
    uint8_t* v_cont;
    int8_t* mean_q;
    float* mean_scale;
    uint32_t* status;
    int T, Hkv, max_windows, mean_mode, do_k, do_v;
    const float* rope_cos;   // [positions][64], nullable: keys are handed over before their rotary embedding
    const float* rope_sin;
    int rope_style;          // 0 none, DQ_ROPE_HALF, DQ_ROPE_PAIRS
    // Decode-step mode (dq_decode_step): token t is the newest token of sequence t, at position
    // step_seq_lens[t] - 1 (sequences of length 0 have none); seq_id / pos are not read.
    const int32_t* step_seq_lens;
    int* step_flags;         // decode-step mode: 4 hand-over words this kernel clears for the kernels after it
};
// pk / pv: pair alphabets of the key / value table (read only when that table has dev.pair set)
cudaError_t dq_launch_encode(const DqDevTable& tk, const DqDevTable& tv, const DqPairEnc& pk, const DqPairEnc& pv,
                             const DqEncodeArgs& a, cudaStream_t st);
cudaError_t dq_launch_decode_tokens(const DqDevTable& t, const uint8_t* cont, const int8_t* mean_q,
                                    const float* mean_scale, int max_windows, const int32_t* seq_id,
                                    const int32_t* pos, const int32_t* slot, int T, int Hkv,
                                    uint8_t* symbols, float* dequant, cudaStream_t st);

cudaError_t dq_launch_window_append(const void* k_new, const void* v_new, void* resid_k, void* resid_v,
                                    int32_t* resid_lens, int cap, int B, int Hkv, cudaStream_t st);

struct DqAttnArgs {
    const void* q_bf16;
    const uint8_t* k_cont;
    const uint8_t* v_cont;
    const int8_t* mean_q;
    const float* mean_scale;
    const int32_t* page_table;
    const int32_t* seq_lens;
    void* out_bf16;
    float* out_f32;
    void* workspace;
    int max_windows, max_pages, B, Hq, Hkv;
    float sm_scale;
    const void* resid_k;        // bf16 [B][resid_cap][Hkv][128], nullable
    const void* resid_v;
    const int32_t* resid_lens;  // [B]
    int resid_cap;
    int q_len;                  // query tokens per sequence (q and out are [B][q_len][Hq][128]); 0 or 1: one
    int fused;                  // decode-step mode: launched right after the step's encoder (see dq_decode_step)
};
size_t dq_attn_workspace_bytes(int B, int Hq, int max_pages);
int* dq_attn_workspace_flags(void* workspace);   // the 4 scheduling / hand-over words at the head of a workspace
cudaError_t dq_launch_step(const DqDevTable& tk, const DqDevTable& tv, const DqEncodeArgs& enc, const DqAttnArgs& a,
                           cudaStream_t st);   // encode -> prepare -> attention -> combine
cudaError_t dq_launch_attention(const DqDevTable& tk, const DqDevTable& tv, const DqAttnArgs& a,
                                cudaStream_t st);
cudaError_t dq_attn_static_scratch(void** out);
cudaError_t dq_launch_attention_static(const DqDevTable& tk, const DqDevTable& tv, const DqAttnArgs& a,
                                       cudaStream_t st);
void dq_attn_profile_enable(int on);
int dq_attn_profile_read(float* ms, int max_records);
cudaError_t dq_launch_bf16_attention(const DqAttnArgs& a, const void* k_pages, const void* v_pages,
                                     cudaStream_t st);

// dq_microbench.cu: bare decode loop (measurement aid)
cudaError_t dq_launch_microbench_decode_loop(const DqDevTable& t, const uint8_t* bytes, size_t nbytes, int ctas, int threads,
                                             int chains, int reps, uint32_t* out, cudaStream_t st);
