// Declarations shared by the decode-attention translation units: kernel parameters, the
// layout constants of the workspace records, and a few device helpers.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "dq_device.cuh"
#include "dq_internal.h"

namespace dqattn {

constexpr int kN = DQ_HEAD_DIM;
constexpr int kChunk = 32;             // tokens per warp per item
constexpr int kQ16Stride = 272;        // bytes per row of the fp16 q' operand (128 halves + pad)
constexpr int kQ16Bytes = 16 * kQ16Stride;
constexpr int kPartial = 132;          // floats per partial record: 128 acc, m, l, off, pad
constexpr int kORow = 132;             // floats per head row of a warp's output slot
constexpr int kMaxWarps = 16;

struct AttnParams {
    const uint16_t* q;
    const uint8_t* k_cont;
    const uint8_t* v_cont;
    const int8_t* mean_q;
    const float* mean_scale;
    const int32_t* page_table;
    const int32_t* seq_lens;
    int* counter;
    int* prefix;        // [B + 1] blocks before sequence b
    float* qrot;        // [B][Hq][128]              rotated q (bf16 baseline reads q itself)
    uint16_t* q16;      // [B][Hkv][16][128] halves  fp16 hi (rows g) / lo (rows 8 + g) of q'
    float* qsum;        // [B][Hq]                   sum_j q'_j
    float* qmu;         // [B][Hq][windows]          sum_j q'_j mean_j of every window
    float* partial;     // [blocks][Hq][kPartial]
    void* out_bf16;
    float* out_f32;
    int max_windows, windows, max_pages, B, Hq, Hkv, G, item_tokens, rotate_q, rotate_out, has_mean;
    float scale_log2;   // sm_scale * log2(e)
    unsigned hkv_magic; // ceil(2^32 / Hkv), 0 when Hkv = 1 (token-wide streams: of Hkv / hs)
    int hs, groups;     // heads per stream, streams per token (Hkv / hs); per-head tables: 1, Hkv
    // Several query tokens per sequence (q_len > 1): the rows of one KV head are (query token i, head g),
    // r = i * G1 + g; G = q_len * G1 rows per KV head and Hq = Hkv * G rows per sequence everywhere in the
    // workspace.  Query token i is q_len - 1 - i positions before the end of the sequence.
    int q_len, G1, Hq1; // query tokens of this pass; query heads per KV head and per token
    // Decode-step mode (dq_decode_step): the attention kernel starts while the step's encoder still runs.
    // flags: [0] next dynamic item, [1] set when the prepare kernel's outputs are complete, [2] prepare
    // CTAs finished, [3] times a CTA gave up polling [1].  ne_before[b]: non-empty sequences before b.
    int fused, attn_grid;
    int poll_limit;   // decode-step mode: polls of the ready flag before a CTA falls back to the grid dependency wait
    int* flags;
    int* ne_before;
    int q_total, q_first; // tokens per sequence in q / out, and the first one this pass handles (a call with
                        // more rows than one MMA tile holds is run as several passes)
    const uint16_t* resid_k;      // bf16 [B][resid_cap][Hkv][128], nullable: uncompressed recent tokens
    const uint16_t* resid_v;
    const int32_t* resid_lens;    // [B]
    int resid_cap;
};

__device__ __forceinline__ uint32_t dp4a_u32(uint32_t a, uint32_t b, uint32_t c) {
    uint32_t d;
    asm("dp4a.u32.u32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}

__device__ __forceinline__ uint32_t pack_half2(float a, float b) {
    const __half2 h = __floats2half2_rn(a, b);
    return *reinterpret_cast<const uint32_t*>(&h);
}

// 2^x for x <= 0 (softmax weights): one MUFU; results below 2^-126 flush to zero, 2^-inf = 0.
__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ void sts128(uint32_t addr, const uint32_t* v) {
    asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};\n" ::"r"(addr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3])
                 : "memory");
}
__device__ __forceinline__ void sts32f(uint32_t addr, float v) {
    asm volatile("st.shared.f32 [%0], %1;\n" ::"r"(addr), "f"(v) : "memory");
}

// Source / destination of workspace row (b, hq) in q / out, laid out [B][q_total][Hq1][128].
__device__ __forceinline__ size_t qo_row(const AttnParams& p, int b, int hq) {
    const int h = hq / p.G, r = hq - h * p.G, i = r / p.G1, g = r - i * p.G1;
    return ((size_t)b * p.q_total + p.q_first + i) * p.Hq1 + (size_t)h * p.G1 + g;
}
// Positions before the sequence end of the query token that row r of a KV head belongs to.
__device__ __forceinline__ int row_offset(const AttnParams& p, int r) {
    return r < p.G ? p.q_total - 1 - (p.q_first + r / p.G1) : 0;
}

}  // namespace dqattn

// Main kernel of the token-wide path (dq_attention_wide.cu): warps per CTA that fit the
// device's shared memory (0: none do), and the launch itself; prepare / combine are shared.
int dq_attn_wide_pick_warps(const DqDevTable& tk, const DqDevTable& tv, int B, int G, int smem_max);
cudaError_t dq_launch_attention_wide_main(const DqDevTable& tk, const DqDevTable& tv, const dqattn::AttnParams& p,
                                          int nw, int sm_count, cudaStream_t st);
