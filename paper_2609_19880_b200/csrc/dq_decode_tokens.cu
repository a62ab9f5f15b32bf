// Check/debug decoder: Algorithm 2 on every record, one thread per stream, reading the
// record straight from global memory.  Produces the symbols and the dequantised values
// xhat = fma(m, s, o) (+ window mean for keys, Appendix A).  Not a performance path.
#include <cuda_fp16.h>

#include "dq_internal.h"

namespace {

__global__ void __launch_bounds__(128)
dq_decode_tokens_kernel(const __grid_constant__ DqDevTable T, const uint8_t* __restrict__ cont,
                        const int8_t* __restrict__ mean_q, const float* __restrict__ mean_scale,
                        int Wmax, const int32_t* __restrict__ seq_id, const int32_t* __restrict__ pos,
                        const int32_t* __restrict__ slot, int n_tok, int Hkv,
                        uint8_t* __restrict__ symbols, float* __restrict__ dequant) {
    const long long sid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (sid >= (long long)n_tok * Hkv) return;
    const int t = (int)(sid / Hkv), h = (int)(sid % Hkv);
    const int sl = slot[t];
    const uint8_t* rec = cont + (((size_t)(sl / DQ_PAGE_TOKENS) * Hkv + h) * DQ_PAGE_TOKENS +
                                 (size_t)(sl % DQ_PAGE_TOKENS)) * T.rec;
    const float s = __half2float(__ushort_as_half((unsigned short)(rec[0] | (rec[1] << 8))));
    const float o = __half2float(__ushort_as_half((unsigned short)(rec[2] | (rec[3] << 8))));
    // final state: sigma / 8 bytes, little-endian; the state interval starts at L = 2^(sigma - 9)
    uint32_t x = (uint32_t)rec[4] | ((uint32_t)rec[5] << 8) | ((uint32_t)rec[6] << 16);
    if (T.sigma == 32) x |= (uint32_t)rec[7] << 24;
    int ptr = 4 + (T.sigma >> 3);
    const uint32_t L = 1u << (T.sigma - 9);
    const int8_t* mq = nullptr;
    float msc = 0.f;
    if (T.has_mean && mean_q) {
        const size_t mi = ((size_t)seq_id[t] * Wmax + pos[t] / DQ_WINDOW_TOKENS) * Hkv + h;
        mq = mean_q + mi * DQ_HEAD_DIM;
        msc = mean_scale[mi];
    }
    auto emit = [&](int j, float lvl) {
        if (symbols) symbols[sid * DQ_HEAD_DIM + j] = (uint8_t)(int)lvl;
        if (dequant) {
            float v = __fmaf_rn(lvl, s, o);
            if (mq) v = __fadd_rn(v, __fmul_rn(msc, (float)mq[j]));
            dequant[sid * DQ_HEAD_DIM + j] = v;
        }
    };
    if (T.pair) {   // one step per pair of values: entry = code(b) << 24 | f << 16 | code(a) << 8 | (z - c)
        for (int j = 0; j < DQ_HEAD_DIM; j += 2) {
            const uint32_t e = T.lut[x & 255u];
            x = ((e >> 16) & 255u) * (x >> 8) + (e & 255u);
            if (x < L && ptr < T.rec) x = (x << 8) | rec[ptr++];  // at most one byte
            emit(j, __half2float(__ushort_as_half((unsigned short)(e & 0xff00u))));
            emit(j + 1, __half2float(__ushort_as_half((unsigned short)((e >> 16) & 0xff00u))));
        }
        return;
    }
    for (int j = 0; j < DQ_HEAD_DIM; ++j) {
        const uint32_t e = T.lut[x & 255u];
        x = (e >> 24) * (x >> 8) + (e & 255u);
        if (x < L && ptr < T.rec) x = (x << 8) | rec[ptr++];  // at most one byte
        emit(j, __half2float(__ushort_as_half((unsigned short)((e >> 8) & 0xffffu))));
    }
}

// Token-wide streams: one thread per (token, group of hs heads), record read from the
// word-interleaved page layout; symbols / dequantised values are written per head.
__global__ void __launch_bounds__(128)
dq_decode_tokens_wide_kernel(const __grid_constant__ DqDevTable T, const uint8_t* __restrict__ cont,
                             const int8_t* __restrict__ mean_q, const float* __restrict__ mean_scale,
                             int Wmax, const int32_t* __restrict__ seq_id, const int32_t* __restrict__ pos,
                             const int32_t* __restrict__ slot, int n_tok, int Hkv,
                             uint8_t* __restrict__ symbols, float* __restrict__ dequant) {
    const int groups = Hkv / T.hs;
    const long long sid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (sid >= (long long)n_tok * groups) return;
    const int t = (int)(sid / groups), grp = (int)(sid % groups);
    const int sl = slot[t];
    const uint8_t* blk = cont + ((size_t)(sl / DQ_PAGE_TOKENS) * groups + grp) * ((size_t)T.rec_words * 64) +
                         (size_t)(sl % DQ_PAGE_TOKENS) * 4;
    auto byte_at = [&](int i) -> uint32_t { return blk[(size_t)(i >> 2) * 64 + (i & 3)]; };
    const float s = __half2float(__ushort_as_half((unsigned short)(byte_at(0) | (byte_at(1) << 8))));
    const float o = __half2float(__ushort_as_half((unsigned short)(byte_at(2) | (byte_at(3) << 8))));
    uint32_t x = byte_at(4) | (byte_at(5) << 8) | (byte_at(6) << 16) | (byte_at(7) << 24);
    int ptr = 8;
    for (int k = 0; k < T.hs; ++k) {
        const int h = grp * T.hs + k;
        const int8_t* mq = nullptr;
        float msc = 0.f;
        if (T.has_mean && mean_q) {
            const size_t mi = ((size_t)seq_id[t] * Wmax + pos[t] / DQ_WINDOW_TOKENS) * Hkv + h;
            mq = mean_q + mi * DQ_HEAD_DIM;
            msc = mean_scale[mi];
        }
        const size_t dst = ((size_t)t * Hkv + h) * DQ_HEAD_DIM;
        auto emit = [&](int j, float lvl) {
            if (symbols) symbols[dst + j] = (uint8_t)(int)lvl;
            if (dequant) {
                float v = __fmaf_rn(lvl, s, o);
                if (mq) v = __fadd_rn(v, __fmul_rn(msc, (float)mq[j]));
                dequant[dst + j] = v;
            }
        };
        if (T.pair) {   // one step per pair of values: entry = code(b) << 24 | f << 16 | code(a) << 8 | (z - c)
            for (int j = 0; j < DQ_HEAD_DIM; j += 2) {
                const uint32_t e = T.lut[x & 255u];
                x = ((e >> 16) & 255u) * (x >> 8) + (e & 255u);
                if (x < (1u << 23) && ptr < T.rec) x = (x << 8) | byte_at(ptr++);
                emit(j, __half2float(__ushort_as_half((unsigned short)(e & 0xff00u))));
                emit(j + 1, __half2float(__ushort_as_half((unsigned short)((e >> 16) & 0xff00u))));
            }
            continue;
        }
        for (int j = 0; j < DQ_HEAD_DIM; ++j) {
            const uint32_t e = T.lut[x & 255u];
            x = (e >> 24) * (x >> 8) + (e & 255u);
            if (x < (1u << 23) && ptr < T.rec) x = (x << 8) | byte_at(ptr++);
            emit(j, __half2float(__ushort_as_half((unsigned short)((e >> 8) & 0xffffu))));
        }
    }
}

// BF16 residual window (Sec. 5.1: the most recent tokens stay uncompressed): append one new
// token per sequence at position resid_lens[b] and count it.  One CTA per sequence; a full
// window is left unchanged.
__global__ void __launch_bounds__(256)
dq_window_append_kernel(const uint4* __restrict__ k_new, const uint4* __restrict__ v_new, uint4* __restrict__ resid_k,
                        uint4* __restrict__ resid_v, int32_t* __restrict__ resid_lens, int cap, int Hkv) {
    const int b = blockIdx.x;
    const int r = resid_lens[b];
    __syncthreads();   // every thread has read the count before thread 0 advances it
    if (r < 0 || r >= cap) return;
    const int row16 = Hkv * (DQ_HEAD_DIM * 2 / 16);   // 16-byte pieces of one token's K (or V)
    const size_t dst = ((size_t)b * cap + r) * row16, src = (size_t)b * row16;
    for (int i = threadIdx.x; i < row16; i += blockDim.x) {
        resid_k[dst + i] = k_new[src + i];
        resid_v[dst + i] = v_new[src + i];
    }
    if (threadIdx.x == 0) resid_lens[b] = r + 1;
}

}  // namespace

cudaError_t dq_launch_window_append(const void* k_new, const void* v_new, void* resid_k, void* resid_v,
                                    int32_t* resid_lens, int cap, int B, int Hkv, cudaStream_t st) {
    if (B == 0) return cudaSuccess;
    dq_window_append_kernel<<<B, 256, 0, st>>>(static_cast<const uint4*>(k_new), static_cast<const uint4*>(v_new),
                                               static_cast<uint4*>(resid_k), static_cast<uint4*>(resid_v), resid_lens,
                                               cap, Hkv);
    return cudaGetLastError();
}

cudaError_t dq_launch_decode_tokens(const DqDevTable& t, const uint8_t* cont, const int8_t* mean_q,
                                    const float* mean_scale, int max_windows, const int32_t* seq_id,
                                    const int32_t* pos, const int32_t* slot, int T, int Hkv,
                                    uint8_t* symbols, float* dequant, cudaStream_t st) {
    if (t.hs > 1) {
        const long long ns = (long long)T * (Hkv / t.hs);
        if (ns == 0) return cudaSuccess;
        dq_decode_tokens_wide_kernel<<<(unsigned)((ns + 127) / 128), 128, 0, st>>>(
            t, cont, mean_q, mean_scale, max_windows, seq_id, pos, slot, T, Hkv, symbols, dequant);
        return cudaGetLastError();
    }
    const long long n = (long long)T * Hkv;
    if (n == 0) return cudaSuccess;
    dq_decode_tokens_kernel<<<(unsigned)((n + 127) / 128), 128, 0, st>>>(
        t, cont, mean_q, mean_scale, max_windows, seq_id, pos, slot, T, Hkv, symbols, dequant);
    return cudaGetLastError();
}
