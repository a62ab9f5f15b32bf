// Encoder kernels: window means of keys and the one-warp-per-stream encoder
// (Fig. 1 pipeline; Algorithm 1; Sec. 4.5 "Encoding").  Compiled with -fmad=false: every
// floating-point operation below is a single IEEE operation in a fixed order so that the
// records are reproducible bit for bit.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "dq_device.cuh"
#include "dq_internal.h"

namespace {

constexpr unsigned kFull = dqdev::kFullMask;
constexpr int kN = DQ_HEAD_DIM;
constexpr uint32_t kL = 1u << 23;  // lower bound of the rANS state interval

using dqdev::bf16_bits_to_float;
using dqdev::warp_fwht128;  // per-head Hadamard rotation (Sec. 4.2), 4 values per lane

// ------------------------------------------------------------------ window means

// DQ_MEAN_COMPUTE.  A run is a maximal range of consecutive call tokens with the same
// (seq_id, pos / 128).  One warp per (run head token, KV head); warps whose token is not
// the first of its run exit.  Sequential binary32 sum over the run, times 1/count, rotated,
// quantised to INT8 with one scale (max |mean| / 127).
__global__ void __launch_bounds__(256)
dq_means_compute_kernel(const uint16_t* __restrict__ k, int T, int Hkv, int rotate,
                        const int32_t* __restrict__ seq_id, const int32_t* __restrict__ pos,
                        int8_t* __restrict__ mean_q, float* __restrict__ mean_scale, int Wmax) {
    const int lane = threadIdx.x & 31;
    const long long wid = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (wid >= (long long)T * Hkv) return;
    const int t0 = (int)(wid / Hkv), h = (int)(wid % Hkv);
    const int s = seq_id[t0], w = pos[t0] / DQ_WINDOW_TOKENS;
    if (t0 > 0 && seq_id[t0 - 1] == s && pos[t0 - 1] / DQ_WINDOW_TOKENS == w) return;
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    int t = t0;
    for (; t < T; ++t) {
        if (t > t0 && !(seq_id[t] == s && pos[t] / DQ_WINDOW_TOKENS == w)) break;
        const uint2 raw = *reinterpret_cast<const uint2*>(k + ((size_t)t * Hkv + h) * kN + 4 * lane);
        acc[0] = __fadd_rn(acc[0], bf16_bits_to_float(raw.x & 0xffffu));
        acc[1] = __fadd_rn(acc[1], bf16_bits_to_float(raw.x >> 16));
        acc[2] = __fadd_rn(acc[2], bf16_bits_to_float(raw.y & 0xffffu));
        acc[3] = __fadd_rn(acc[3], bf16_bits_to_float(raw.y >> 16));
    }
    const float inv = __fdiv_rn(1.0f, (float)(t - t0));
#pragma unroll
    for (int e = 0; e < 4; ++e) acc[e] = __fmul_rn(acc[e], inv);
    if (rotate) warp_fwht128(acc, lane);
    float amax = fmaxf(fmaxf(fabsf(acc[0]), fabsf(acc[1])), fmaxf(fabsf(acc[2]), fabsf(acc[3])));
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) amax = fmaxf(amax, __shfl_xor_sync(kFull, amax, d));
    const float sc = __fdiv_rn(amax, 127.0f);
    uint32_t packed = 0;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        float q = 0.f;
        if (sc != 0.f) q = fminf(fmaxf(rintf(__fdiv_rn(acc[e], sc)), -127.f), 127.f);
        packed |= ((uint32_t)(int)q & 0xffu) << (8 * e);
    }
    const size_t mi = ((size_t)s * Wmax + w) * Hkv + h;
    *reinterpret_cast<uint32_t*>(mean_q + mi * kN + 4 * lane) = packed;
    if (lane == 0) mean_scale[mi] = sc;
}

// DQ_MEAN_REUSE.  A token at the first position of a window copies the previous window's
// mean into its own (window 0: zeros).  One warp per (token, KV head).
__global__ void __launch_bounds__(256)
dq_means_reuse_kernel(int T, int Hkv, const int32_t* __restrict__ seq_id,
                      const int32_t* __restrict__ pos, int8_t* __restrict__ mean_q,
                      float* __restrict__ mean_scale, int Wmax) {
    const int lane = threadIdx.x & 31;
    const long long wid = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (wid >= (long long)T * Hkv) return;
    const int t = (int)(wid / Hkv), h = (int)(wid % Hkv);
    const int p = pos[t];
    if (p % DQ_WINDOW_TOKENS) return;
    const int w = p / DQ_WINDOW_TOKENS;
    const size_t dst = ((size_t)seq_id[t] * Wmax + w) * Hkv + h;
    uint32_t q = 0;
    float sc = 0.f;
    if (w > 0) {
        const size_t src = ((size_t)seq_id[t] * Wmax + (w - 1)) * Hkv + h;
        q = *reinterpret_cast<const uint32_t*>(mean_q + src * kN + 4 * lane);
        sc = mean_scale[src];
    }
    *reinterpret_cast<uint32_t*>(mean_q + dst * kN + 4 * lane) = q;
    if (lane == 0) mean_scale[dst] = sc;
}

// ------------------------------------------------------------------------ drift

// Function Drift of Algorithm 1 on a stream held 4 values per lane.  The bisection of
// log2(lambda) over T = 12 steps is carried out as the geometric mean of the bracket
// [hi * 2^-40, hi], hi = 8 (max D - min D); the code length is an integer sum of
// ceil(65536 r_m), so the feasibility test does not depend on summation order.
// Returns the length of the final assignment (the argmin at the bracket's upper end).
__device__ __forceinline__ uint32_t drift(const DqDevTable& T, const float (&z)[4], float s, float o,
                                          uint32_t (&sym)[4]) {
    const int M = T.M;
    float maxD = -INFINITY, minD = INFINITY;
    for (int m = 0; m < M; ++m) {
        const float tm = __fmaf_rn((float)m, s, o);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float d = __fsub_rn(z[e], tm);
            const float D = __fmul_rn(d, d);
            maxD = fmaxf(maxD, D);
            minD = fminf(minD, D);
        }
    }
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) {
        maxD = fmaxf(maxD, __shfl_xor_sync(kFull, maxD, d));
        minD = fminf(minD, __shfl_xor_sync(kFull, minD, d));
    }
    const uint32_t budget = (uint32_t)T.budget_bits << 16;
    float lam_hi = __fmul_rn(8.0f, __fsub_rn(maxD, minD));
    float lam_lo = __fmul_rn(lam_hi, 0x1p-40f);
    uint32_t len = 0;
    for (int it = 0; it <= 12; ++it) {
        const float lam = (it < 12) ? __fsqrt_rn(__fmul_rn(lam_lo, lam_hi)) : lam_hi;
        float best[4];
        uint32_t cost_fx[4];
        for (int m = 0; m < M; ++m) {
            const float tm = __fmaf_rn((float)m, s, o);
            const float rm = T.r[m];
            const uint32_t Rm = T.R[m];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float d = __fsub_rn(z[e], tm);
                const float c = __fmaf_rn(lam, rm, __fmul_rn(d, d));
                if (m == 0 || c < best[e]) { best[e] = c; sym[e] = (uint32_t)m; cost_fx[e] = Rm; }
            }
        }
        len = __reduce_add_sync(kFull, cost_fx[0] + cost_fx[1] + cost_fx[2] + cost_fx[3]);
        if (it < 12) {
            if (len <= budget) lam_hi = lam; else lam_lo = lam;
        }
    }
    return len;
}

// ---------------------------------------------------------------------- encoder

constexpr int kEncWarps = 8;

// One warp per stream (token, KV head).  Lane l owns elements 4l .. 4l+3.
__global__ void __launch_bounds__(kEncWarps * 32)
dq_encode_kernel(const __grid_constant__ DqDevTable T, const uint16_t* __restrict__ x, int n_tok,
                 int Hkv, const int32_t* __restrict__ seq_id, const int32_t* __restrict__ pos,
                 const int32_t* __restrict__ slot, uint8_t* __restrict__ cont,
                 const int8_t* __restrict__ mean_q, const float* __restrict__ mean_scale, int Wmax,
                 uint32_t* __restrict__ status) {
    __shared__ uint8_t s_bytes[kEncWarps][DQ_MAX_REC_BYTES];
    const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
    const long long wid = (long long)blockIdx.x * kEncWarps + wib;
    if (wid >= (long long)n_tok * Hkv) return;
    const int t = (int)(wid / Hkv), h = (int)(wid % Hkv);

    float z[4];
    {
        const uint2 raw = *reinterpret_cast<const uint2*>(x + ((size_t)t * Hkv + h) * kN + 4 * lane);
        z[0] = bf16_bits_to_float(raw.x & 0xffffu); z[1] = bf16_bits_to_float(raw.x >> 16);
        z[2] = bf16_bits_to_float(raw.y & 0xffffu); z[3] = bf16_bits_to_float(raw.y >> 16);
    }
    if (T.rotate) warp_fwht128(z, lane);
    if (T.has_mean) {  // remove the (dequantised) windowed channel mean, Sec. 4.2
        const size_t mi = ((size_t)seq_id[t] * Wmax + pos[t] / DQ_WINDOW_TOKENS) * Hkv + h;
        const float sc = mean_scale[mi];
        const uint32_t q4 = *reinterpret_cast<const uint32_t*>(mean_q + mi * kN + 4 * lane);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float q = (float)(int)(int8_t)((q4 >> (8 * e)) & 0xffu);
            z[e] = __fsub_rn(z[e], __fmul_rn(sc, q));
        }
    }
    float mx = fmaxf(fmaxf(z[0], z[1]), fmaxf(z[2], z[3]));
    float mn = fminf(fminf(z[0], z[1]), fminf(z[2], z[3]));
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) {
        mx = fmaxf(mx, __shfl_xor_sync(kFull, mx, d));
        mn = fminf(mn, __shfl_xor_sync(kFull, mn, d));
    }

    uint32_t sym[4];
    __half s16 = __ushort_as_half(0), o16 = __ushort_as_half(0);
    bool degenerate = !(mx > mn);
    uint32_t st_fallback = 0, st_refit = 0;
    if (!degenerate) {
        const float o = mn;                                         // FitMinMax, Eq. (affine_token)
        const float s = __fdiv_rn(__fsub_rn(mx, mn), (float)(T.M - 1));
        drift(T, z, s, o, sym);
        // Refit: least squares of z on the symbols; binary64 sums in a fixed order
        double a = (double)z[0], b = __dmul_rn((double)sym[0], (double)z[0]);
        int sm = (int)sym[0], smm = (int)(sym[0] * sym[0]);
#pragma unroll
        for (int e = 1; e < 4; ++e) {
            a = __dadd_rn(a, (double)z[e]);
            b = __dadd_rn(b, __dmul_rn((double)sym[e], (double)z[e]));
            sm += (int)sym[e];
            smm += (int)(sym[e] * sym[e]);
        }
#pragma unroll
        for (int d = 16; d >= 1; d >>= 1) {
            a = __dadd_rn(a, __shfl_xor_sync(kFull, a, d));
            b = __dadd_rn(b, __shfl_xor_sync(kFull, b, d));
        }
        const long long Sm = __reduce_add_sync(kFull, sm), Smm = __reduce_add_sync(kFull, smm);
        const long long den = (long long)kN * Smm - Sm * Sm;
        double sd = (double)s, od = (double)o;
        if (den != 0) {
            sd = __ddiv_rn(__dsub_rn(__dmul_rn((double)kN, b), __dmul_rn((double)Sm, a)), (double)den);
            od = __ddiv_rn(__dsub_rn(a, __dmul_rn(sd, (double)Sm)), (double)kN);
        }
        s16 = __double2half(sd);                                    // fp16 metadata
        o16 = __double2half(od);
        float sf = __half2float(s16), of = __half2float(o16);
        if (!(isfinite(sf) && sf > 0.0f && isfinite(of))) {
            s16 = __float2half_rn(s);
            o16 = __float2half_rn(o);
            sf = __half2float(s16); of = __half2float(o16);
            st_refit = 1;
        }
        if (!(sf > 0.0f)) degenerate = true;
        else {
            const uint32_t len = drift(T, z, sf, of, sym);          // second Drift, fp16 grid
            if (len > ((uint32_t)T.budget_bits << 16)) {
#pragma unroll
                for (int e = 0; e < 4; ++e) sym[e] = (uint32_t)T.mstar;
                st_fallback = 1;
            }
        }
    }
    if (degenerate) {
        s16 = __ushort_as_half(0);
        o16 = __float2half_rn(mn);
#pragma unroll
        for (int e = 0; e < 4; ++e) sym[e] = (uint32_t)T.mstar;
    }

    // rANS, Eq. (rans) Enc on symbols 127 .. 0 so that decoding runs forward.  Every lane
    // carries the same state; lane 0 records the emitted bytes.
    const uint32_t sym4 = sym[0] | (sym[1] << 8) | (sym[2] << 16) | (sym[3] << 24);
    uint32_t xs = kL;
    int k = 0;
    uint8_t* bytes = s_bytes[wib];
    for (int j = kN - 1; j >= 0; --j) {
        const uint32_t word = __shfl_sync(kFull, sym4, j >> 2);
        const uint32_t m = (word >> (8 * (j & 3))) & 0xffu;
        const uint32_t fc = T.fc[m];
        const uint32_t f = fc & 0xffffu, c = fc >> 16;
        if (xs >= (f << 23)) {  // at most once: xs < 2^31 <= 2^8 * (f << 23)
            if (lane == 0) bytes[k] = (uint8_t)(xs & 0xffu);
            ++k;
            xs >>= 8;
        }
        xs = (xs / f) * 256u + (xs % f) + c;
    }
    __syncwarp();
    const uint32_t hdr0 = (uint32_t)__half_as_ushort(s16) | ((uint32_t)__half_as_ushort(o16) << 16);
    const int sl = slot[t];
    uint8_t* rec = cont + (((size_t)(sl / DQ_PAGE_TOKENS) * Hkv + h) * DQ_PAGE_TOKENS +
                           (size_t)(sl % DQ_PAGE_TOKENS)) * T.rec;
    const int used = min(8 + k, T.rec);  // the budget test keeps 8 + k <= rec
    for (int i = lane; i < T.rec; i += 32) {
        uint8_t v = 0;
        if (i < 4) v = (uint8_t)(hdr0 >> (8 * i));
        else if (i < 8) v = (uint8_t)(xs >> (8 * (i - 4)));
        else if (i < used) v = bytes[k - 1 - (i - 8)];
        rec[i] = v;
    }
    if (status && lane == 0) {
        if (st_fallback) atomicAdd(status + 0, 1u);
        if (degenerate) atomicAdd(status + 1, 1u);
        if (st_refit) atomicAdd(status + 2, 1u);
        atomicMax(status + 3, (uint32_t)(8 + k));
    }
}

}  // namespace

cudaError_t dq_launch_means(const DqDevTable& tk, const void* k_bf16, int T, int Hkv,
                            const int32_t* seq_id, const int32_t* pos, int8_t* mean_q,
                            float* mean_scale, int max_windows, int mode, cudaStream_t st) {
    const long long warps = (long long)T * Hkv;
    if (warps == 0) return cudaSuccess;
    const unsigned blocks = (unsigned)((warps + 7) / 8);
    if (mode == DQ_MEAN_COMPUTE)
        dq_means_compute_kernel<<<blocks, 256, 0, st>>>((const uint16_t*)k_bf16, T, Hkv, tk.rotate,
                                                        seq_id, pos, mean_q, mean_scale, max_windows);
    else
        dq_means_reuse_kernel<<<blocks, 256, 0, st>>>(T, Hkv, seq_id, pos, mean_q, mean_scale,
                                                      max_windows);
    return cudaGetLastError();
}

cudaError_t dq_launch_encode(const DqDevTable& t, const void* x_bf16, int T, int Hkv,
                             const int32_t* seq_id, const int32_t* pos, const int32_t* slot,
                             uint8_t* cont, const int8_t* mean_q, const float* mean_scale,
                             int max_windows, uint32_t* status, cudaStream_t st) {
    const long long warps = (long long)T * Hkv;
    if (warps == 0) return cudaSuccess;
    const unsigned blocks = (unsigned)((warps + kEncWarps - 1) / kEncWarps);
    dq_encode_kernel<<<blocks, kEncWarps * 32, 0, st>>>(t, (const uint16_t*)x_bf16, T, Hkv, seq_id,
                                                        pos, slot, cont, mean_q, mean_scale,
                                                        max_windows, status);
    return cudaGetLastError();
}
