// Encoder kernels: window means of keys and the one-warp-per-stream encoder
// (Fig. 1 pipeline; Algorithm 1; Sec. 4.5 "Encoding").  Compiled with -fmad=false: every
// floating-point operation below is a single IEEE operation in a fixed order so that the
// records are reproducible bit for bit.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include <cstdlib>

#include "dq_device.cuh"
#include "dq_internal.h"

namespace {

constexpr unsigned kFull = dqdev::kFullMask;
constexpr int kN = DQ_HEAD_DIM;
constexpr uint32_t kL = 1u << 23;  // lower bound of the rANS state interval (sigma = 32; token-wide streams always)

using dqdev::bf16_bits_to_float;
using dqdev::warp_fwht128;  // per-head Hadamard rotation (Sec. 4.2), 4 values per lane

// Rotary position embedding of a head vector held 4 values per lane (element 4 lane + e), in
// binary32 with every product and sum rounded once.  DQ_ROPE_HALF pairs element j with j + 64
// (the partner sits in lane ^ 16), DQ_ROPE_PAIRS pairs 2j with 2j + 1 (same lane).
// cs / sn: this position's 64 cosines / sines.
__device__ __forceinline__ void warp_rope128(float (&v)[4], int lane, const float* cs, const float* sn, int style) {
    if (style == DQ_ROPE_HALF) {
        const float4 c = *reinterpret_cast<const float4*>(cs + 4 * (lane & 15));
        const float4 s = *reinterpret_cast<const float4*>(sn + 4 * (lane & 15));
        const float cc[4] = {c.x, c.y, c.z, c.w}, ss[4] = {s.x, s.y, s.z, s.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float other = __shfl_xor_sync(kFull, v[e], 16);
            // lanes 0-15 hold a: a cos - b sin; lanes 16-31 hold b: b cos + a sin
            const float mine = __fmul_rn(v[e], cc[e]), cross = __fmul_rn(other, ss[e]);
            v[e] = (lane < 16) ? __fsub_rn(mine, cross) : __fadd_rn(mine, cross);
        }
    } else {
        const float2 c = *reinterpret_cast<const float2*>(cs + 2 * lane);
        const float2 s = *reinterpret_cast<const float2*>(sn + 2 * lane);
        const float a0 = v[0], b0 = v[1], a1 = v[2], b1 = v[3];
        v[0] = __fsub_rn(__fmul_rn(a0, c.x), __fmul_rn(b0, s.x));
        v[1] = __fadd_rn(__fmul_rn(b0, c.x), __fmul_rn(a0, s.x));
        v[2] = __fsub_rn(__fmul_rn(a1, c.y), __fmul_rn(b1, s.y));
        v[3] = __fadd_rn(__fmul_rn(b1, c.y), __fmul_rn(a1, s.y));
    }
}

// ------------------------------------------------------------------ window means

// Mean of the run that starts at call token t0, for KV head h, by one warp.
__device__ __forceinline__ void means_of_run(const uint16_t* __restrict__ k, int T, int Hkv, int rotate,
                                             const int32_t* __restrict__ seq_id, const int32_t* __restrict__ pos,
                                             int8_t* __restrict__ mean_q, float* __restrict__ mean_scale, int Wmax,
                                             const float* __restrict__ rope_cos, const float* __restrict__ rope_sin,
                                             int rope_style, int t0, int h, int lane) {
    const int s = seq_id[t0], w = pos[t0] / DQ_WINDOW_TOKENS;
    // length of the run: 32 candidates per round, lanes in parallel (the sums below stay sequential)
    int cnt = 0;
    for (int base = t0; base < T; base += 32) {
        const int tt = base + lane;
        const bool same = tt < T && seq_id[tt] == s && pos[tt] / DQ_WINDOW_TOKENS == w;
        const unsigned m = __ballot_sync(kFull, same);
        if (m != kFull) { cnt += __ffs((int)~m) - 1; break; }
        cnt += 32;
    }
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    constexpr int kAheadLoads = 8;   // independent loads in flight; the additions keep token order
    for (int tb = t0; tb < t0 + cnt; tb += kAheadLoads) {
        uint2 raw[kAheadLoads];
#pragma unroll
        for (int u = 0; u < kAheadLoads; ++u) {
            const int tt = min(tb + u, t0 + cnt - 1);
            raw[u] = *reinterpret_cast<const uint2*>(k + ((size_t)tt * Hkv + h) * kN + 4 * lane);
        }
#pragma unroll
        for (int u = 0; u < kAheadLoads; ++u) {
            if (tb + u >= t0 + cnt) break;
            float kt[4] = {bf16_bits_to_float(raw[u].x & 0xffffu), bf16_bits_to_float(raw[u].x >> 16),
                           bf16_bits_to_float(raw[u].y & 0xffffu), bf16_bits_to_float(raw[u].y >> 16)};
            if (rope_style)
                warp_rope128(kt, lane, rope_cos + (size_t)pos[tb + u] * 64, rope_sin + (size_t)pos[tb + u] * 64, rope_style);
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[e] = __fadd_rn(acc[e], kt[e]);
        }
    }
    const int t = t0 + cnt;
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

// DQ_MEAN_COMPUTE.  A run is a maximal range of consecutive call tokens with the same
// (seq_id, pos / 128).  A CTA looks at kMeansTokens consecutive call tokens, lists those that
// start a run, and its warps take the (run, KV head) pairs in turn.  Sequential binary32 sum over
// the run, times 1/count, rotated, quantised to INT8 with one scale (max |mean| / 127).
constexpr int kMeansTokens = 128;
__global__ void __launch_bounds__(256)
dq_means_compute_kernel(const uint16_t* __restrict__ k, int T, int Hkv, int rotate,
                        const int32_t* __restrict__ seq_id, const int32_t* __restrict__ pos,
                        int8_t* __restrict__ mean_q, float* __restrict__ mean_scale, int Wmax,
                        const float* __restrict__ rope_cos, const float* __restrict__ rope_sin, int rope_style) {
    __shared__ int s_first[kMeansTokens];
    __shared__ int s_n;
    const int lane = threadIdx.x & 31;
    if (threadIdx.x == 0) s_n = 0;
    __syncthreads();
    {
        const long long tt = (long long)blockIdx.x * kMeansTokens + threadIdx.x;
        if (threadIdx.x < kMeansTokens && tt < T) {
            const int t = (int)tt;
            const bool first = t == 0 || seq_id[t - 1] != seq_id[t] || pos[t - 1] / DQ_WINDOW_TOKENS != pos[t] / DQ_WINDOW_TOKENS;
            if (first) s_first[atomicAdd(&s_n, 1)] = t;
        }
    }
    __syncthreads();
    const int tasks = s_n * Hkv;
    for (int task = threadIdx.x >> 5; task < tasks; task += (int)(blockDim.x >> 5))
        means_of_run(k, T, Hkv, rotate, seq_id, pos, mean_q, mean_scale, Wmax, rope_cos, rope_sin, rope_style,
                     s_first[task / Hkv], task % Hkv, lane);
}

// ------------------------------------------------------------------------ drift

// Per-CTA copy of the table fields the encoder touches (a CTA encodes one tensor kind).
// With the paired-symbol variant the rANS alphabet is the M^2 pairs u = a M + b: the coder's arrays
// (rcp .. thr) and prk then hold the pair alphabet, r / R are not used.
struct EncTable {
    float r[DQ_MAX_LEVELS];
    uint32_t R[DQ_MAX_LEVELS];
    uint32_t rcp[DQ_MAX_PAIRS];    // Eq. rans Enc by reciprocal: floor(x / f) = umulhi(x, rcp) >> rsh
    uint32_t rsh[DQ_MAX_PAIRS];
    uint32_t bias[DQ_MAX_PAIRS];   // c (+ 255 when f = 1)
    uint32_t cmpl[DQ_MAX_PAIRS];   // 2^p - f
    uint32_t thr[DQ_MAX_PAIRS];    // f << (sigma - 9) = f L: renormalise while the state is not below it
    uint2 prk[DQ_MAX_PAIRS];       // pairs: {bits of r_u, ceil(65536 r_u) << 8 | u}
    int M, rec, mstar, budget_bits, has_mean, rotate;
    int early_exit, sigma;         // codec variants: Drift tries its end multiplier first; bits of final state (32 / 24)
    int pair;                      // paired symbols
    uint32_t central;              // the all-central stream's four levels of a lane, one per byte
};

// Table of one tensor kind into shared memory (threads 0 .. DQ_MAX_PAIRS - 1 and thread 0).
__device__ __forceinline__ void load_enc_table(EncTable& T, const DqDevTable& TK, const DqDevTable& TV,
                                               const DqPairEnc& PK, const DqPairEnc& PV, bool is_v) {
    const int pair = is_v ? TV.pair : TK.pair, sigma = is_v ? TV.sigma : TK.sigma;
    const int i = threadIdx.x;
    if (i < DQ_MAX_LEVELS) {
        T.r[i] = is_v ? TV.r[i] : TK.r[i];
        T.R[i] = is_v ? TV.R[i] : TK.R[i];
    }
    if (i < (pair ? DQ_MAX_PAIRS : DQ_MAX_LEVELS)) {
        uint32_t aux;
        if (pair) {
            T.rcp[i] = is_v ? PV.enc_rcp[i] : PK.enc_rcp[i];
            aux = is_v ? PV.enc_aux[i] : PK.enc_aux[i];
            T.prk[i] = make_uint2(__float_as_uint(is_v ? PV.r[i] : PK.r[i]), ((is_v ? PV.R[i] : PK.R[i]) << 8) | (uint32_t)i);
        } else {
            T.rcp[i] = is_v ? TV.enc_rcp[i] : TK.enc_rcp[i];
            aux = is_v ? TV.enc_aux[i] : TK.enc_aux[i];
        }
        T.bias[i] = aux & 1023u;
        T.cmpl[i] = (aux >> 10) & 511u;
        T.rsh[i] = aux >> 19;
        T.thr[i] = (256u - ((aux >> 10) & 511u)) << (sigma - 9);
    }
    if (i == 0) {
        T.M = is_v ? TV.M : TK.M; T.rec = is_v ? TV.rec : TK.rec; T.mstar = is_v ? TV.mstar : TK.mstar;
        T.budget_bits = is_v ? TV.budget_bits : TK.budget_bits;
        T.has_mean = is_v ? TV.has_mean : TK.has_mean; T.rotate = is_v ? TV.rotate : TK.rotate;
        T.early_exit = is_v ? TV.early_exit : TK.early_exit; T.sigma = sigma;
        T.pair = pair;
        const uint32_t ms = (uint32_t)T.mstar, us = (uint32_t)(is_v ? TV.ustar : TK.ustar), M = (uint32_t)T.M;
        T.central = pair ? (us / M) * 0x00010001u + (us % M) * 0x01000100u : ms * 0x01010101u;
    }
}

// Function Drift of Algorithm 1 on a stream held 4 values per lane.  The bisection of
// log2(lambda) over T = 12 steps is carried out as the geometric mean of the bracket
// [hi * 2^-40, hi], hi = 8 (max D - min D); the code length is an integer sum of
// ceil(65536 r_m), so the feasibility test does not depend on summation order.
// Returns the length of the final assignment (the argmin at the bracket's upper end).
// M is a template parameter so that the M candidate costs of a value are independent
// instructions and the table sits in registers; the minimum keeps the lowest index among equal
// costs, exactly as an ascending scan with a strict comparison does.
template <int M>
__device__ __noinline__ uint32_t drift_m(const EncTable& T, float z0, float z1, float z2, float z3, float s, float o,
                                         uint32_t& sym_packed) {
    const float z[4] = {z0, z1, z2, z3};
    float tm[M], rm[M];
    uint32_t Km[M];   // ceil(65536 r_m) << 8 | m: the minimum tree carries one word for length and index
#pragma unroll
    for (int m = 0; m < M; ++m) {
        tm[m] = __fmaf_rn((float)m, s, o);
        rm[m] = T.r[m];
        Km[m] = (T.R[m] << 8) | (uint32_t)m;
    }
    float D[4][M];
    float maxD = -INFINITY, minD = INFINITY;
#pragma unroll
    for (int e = 0; e < 4; ++e)
#pragma unroll
        for (int m = 0; m < M; ++m) {
            const float d = __fsub_rn(z[e], tm[m]);
            D[e][m] = __fmul_rn(d, d);
            maxD = fmaxf(maxD, D[e][m]);
            minD = fminf(minD, D[e][m]);
        }
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) {
        maxD = fmaxf(maxD, __shfl_xor_sync(kFull, maxD, d));
        minD = fminf(minD, __shfl_xor_sync(kFull, minD, d));
    }
    const uint32_t budget = (uint32_t)T.budget_bits << 16;
    float lam_hi = __fmul_rn(8.0f, __fsub_rn(maxD, minD));
    float lam_lo = __fmul_rn(lam_hi, 0x1p-40f);
    uint32_t len = 0, sym[4] = {0u, 0u, 0u, 0u};
    // Early-exit variant: when each of the 12 tests passes, the upper end walks hi <- sqrt(lo hi) twelve
    // times with lo fixed; sweep -1 evaluates that multiplier and ends the search if its assignment fits.
    float lam_e = lam_hi;
    if (T.early_exit)
        for (int i = 0; i < 12; ++i) lam_e = __fsqrt_rn(__fmul_rn(lam_lo, lam_e));
#pragma unroll 1
    for (int it = T.early_exit ? -1 : 0; it <= 12; ++it) {
        const float lam = (it < 0) ? lam_e : (it < 12) ? __fsqrt_rn(__fmul_rn(lam_lo, lam_hi)) : lam_hi;
        uint32_t cost_sum = 0;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            float c[M];
            uint32_t key[M];
#pragma unroll
            for (int m = 0; m < M; ++m) { c[m] = __fmaf_rn(lam, rm[m], D[e][m]); key[m] = Km[m]; }
            // pairwise minimum, the left (lower index) operand wins ties
#pragma unroll
            for (int w = 1; w < M; w <<= 1)
#pragma unroll
                for (int m = 0; m + w < M; m += 2 * w)
                    if (c[m + w] < c[m]) { c[m] = c[m + w]; key[m] = key[m + w]; }
            sym[e] = key[0];
            cost_sum += key[0];
        }
        len = __reduce_add_sync(kFull, cost_sum >> 8);   // four indices (< 16 each) stay below bit 8
        if (it < 0) {
            if (len <= budget) break;
        } else if (it < 12) {
            if (len <= budget) lam_hi = lam; else lam_lo = lam;
        }
    }
    sym_packed = (sym[0] & 0xffu) | ((sym[1] & 0xffu) << 8) | ((sym[2] & 0xffu) << 16) | (sym[3] << 24);
    return len;
}

__device__ __forceinline__ uint32_t drift(const EncTable& T, const float (&z)[4], float s, float o,
                                          uint32_t (&sym)[4]) {
    uint32_t packed = 0, len = 0;
    switch (T.M) {   // uniform across the CTA
#define DQ_DRIFT_CASE(M_) case M_: len = drift_m<M_>(T, z[0], z[1], z[2], z[3], s, o, packed); break;
        DQ_DRIFT_CASE(2) DQ_DRIFT_CASE(3) DQ_DRIFT_CASE(4) DQ_DRIFT_CASE(5) DQ_DRIFT_CASE(6) DQ_DRIFT_CASE(7)
        DQ_DRIFT_CASE(8) DQ_DRIFT_CASE(9) DQ_DRIFT_CASE(10) DQ_DRIFT_CASE(11) DQ_DRIFT_CASE(12) DQ_DRIFT_CASE(13)
        DQ_DRIFT_CASE(14) DQ_DRIFT_CASE(15) DQ_DRIFT_CASE(16)
#undef DQ_DRIFT_CASE
        default: break;
    }
#pragma unroll
    for (int e = 0; e < 4; ++e) sym[e] = (packed >> (8 * e)) & 0xffu;
    return len;
}

// Drift for the paired-symbol variant: a lane's values (0, 1) and (2, 3) are two rANS symbols; each takes
// the pair u = a M + b that minimises (D_a + D_b) + lambda r_u, the lowest u among equal costs (rows a in
// ascending order, each reduced pairwise with the left operand winning ties, a later row replacing the best
// only when strictly cheaper: the same winner as an ascending scan with a strict comparison).  Bracket: hi = 16 (max D - min D), D over single values as above.
template <int M>
__device__ __noinline__ uint32_t drift_pair_m(const EncTable& T, float z0, float z1, float z2, float z3, float s, float o,
                                              uint32_t& sym_packed) {
    const float z[4] = {z0, z1, z2, z3};
    float D[4][M];
    float maxD = -INFINITY, minD = INFINITY;
#pragma unroll
    for (int m = 0; m < M; ++m) {
        const float tm = __fmaf_rn((float)m, s, o);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float d = __fsub_rn(z[e], tm);
            D[e][m] = __fmul_rn(d, d);
            maxD = fmaxf(maxD, D[e][m]);
            minD = fminf(minD, D[e][m]);
        }
    }
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) {
        maxD = fmaxf(maxD, __shfl_xor_sync(kFull, maxD, d));
        minD = fminf(minD, __shfl_xor_sync(kFull, minD, d));
    }
    const uint32_t budget = (uint32_t)T.budget_bits << 16;
    float lam_hi = __fmul_rn(16.0f, __fsub_rn(maxD, minD));
    float lam_lo = __fmul_rn(lam_hi, 0x1p-40f);
    uint32_t len = 0, psym[2] = {0u, 0u};
    float lam_e = lam_hi;
    if (T.early_exit)
        for (int i = 0; i < 12; ++i) lam_e = __fsqrt_rn(__fmul_rn(lam_lo, lam_e));
#pragma unroll 1
    for (int it = T.early_exit ? -1 : 0; it <= 12; ++it) {
        const float lam = (it < 0) ? lam_e : (it < 12) ? __fsqrt_rn(__fmul_rn(lam_lo, lam_hi)) : lam_hi;
        uint32_t cost_sum = 0;
#pragma unroll
        for (int p = 0; p < 2; ++p) {
            float rc[M];
            uint32_t rkey[M];
#pragma unroll
            for (int a = 0; a < M; ++a) {
                float c[M];
                uint32_t key[M];
#pragma unroll
                for (int b = 0; b < M; ++b) {
                    const uint2 e = T.prk[a * M + b];
                    c[b] = __fmaf_rn(lam, __uint_as_float(e.x), __fadd_rn(D[2 * p][a], D[2 * p + 1][b]));
                    key[b] = e.y;
                }
#pragma unroll
                for (int w = 1; w < M; w <<= 1)
#pragma unroll
                    for (int b = 0; b + w < M; b += 2 * w)
                        if (c[b + w] < c[b]) { c[b] = c[b + w]; key[b] = key[b + w]; }
                rc[a] = c[0];
                rkey[a] = key[0];
            }
#pragma unroll
            for (int w = 1; w < M; w <<= 1)   // row winners, the left (lower a) operand wins ties
#pragma unroll
                for (int a = 0; a + w < M; a += 2 * w)
                    if (rc[a + w] < rc[a]) { rc[a] = rc[a + w]; rkey[a] = rkey[a + w]; }
            psym[p] = rkey[0];
            cost_sum += rkey[0];
        }
        len = __reduce_add_sync(kFull, cost_sum >> 8);   // two pair indices (< 81 each) stay below bit 8
        if (it < 0) {
            if (len <= budget) break;
        } else if (it < 12) {
            if (len <= budget) lam_hi = lam; else lam_lo = lam;
        }
    }
    const uint32_t u0 = psym[0] & 0xffu, u1 = psym[1] & 0xffu;
    sym_packed = (u0 / M) | ((u0 % M) << 8) | ((u1 / M) << 16) | ((u1 % M) << 24);
    return len;
}

__device__ __forceinline__ uint32_t drift_pair(const EncTable& T, const float (&z)[4], float s, float o,
                                               uint32_t (&sym)[4]) {
    uint32_t packed = 0, len = 0;
    switch (T.M) {   // uniform across the CTA
#define DQ_DRIFT_CASE(M_) case M_: len = drift_pair_m<M_>(T, z[0], z[1], z[2], z[3], s, o, packed); break;
        DQ_DRIFT_CASE(2) DQ_DRIFT_CASE(3) DQ_DRIFT_CASE(4) DQ_DRIFT_CASE(5) DQ_DRIFT_CASE(6) DQ_DRIFT_CASE(7)
        DQ_DRIFT_CASE(8) DQ_DRIFT_CASE(9)
#undef DQ_DRIFT_CASE
        default: break;
    }
#pragma unroll
    for (int e = 0; e < 4; ++e) sym[e] = (packed >> (8 * e)) & 0xffu;
    return len;
}

// ---------------------------------------------------------------------- encoder

constexpr int kEncWarps = 8;
#ifndef DQ_STEP_ENC_WARPS
#define DQ_STEP_ENC_WARPS 16
#endif

// Position and sequence of call token t (decode-step mode derives them from the sequence lengths).
__device__ __forceinline__ int tok_pos(const DqEncodeArgs& a, int t) { return a.step_seq_lens ? a.step_seq_lens[t] - 1 : a.pos[t]; }
__device__ __forceinline__ int tok_seq(const DqEncodeArgs& a, int t) { return a.step_seq_lens ? t : a.seq_id[t]; }

struct StreamQuantised {
    uint32_t hdr0;      // s fp16 | o fp16 << 16
    uint32_t flags;     // 1: all-central fallback, 2: constant stream, 4: refit rejected
    uint32_t sym;       // this lane's four symbols, one per byte
};

// Steps 1-6 of Algorithm 1 for the stream (token t, KV head h) by one warp: rotation (and rotary
// embedding when asked), mean removal, min-max grid, drift, refit, fp16 metadata, second drift.
// PAIR: the table's rANS symbols are pairs of levels (a kernel instantiation of its own, so that the
// single-level kernels carry none of its code).
template <bool PAIR>
__device__ __forceinline__ StreamQuantised quantise_stream(const EncTable& T, const DqEncodeArgs& a, bool is_v, int t, int h,
                                                           int lane) {
    const int Hkv = a.Hkv;
    const uint16_t* x = static_cast<const uint16_t*>(is_v ? a.v_bf16 : a.k_bf16);
    float z[4];
    {
        const uint2 raw = *reinterpret_cast<const uint2*>(x + ((size_t)t * Hkv + h) * kN + 4 * lane);
        z[0] = bf16_bits_to_float(raw.x & 0xffffu); z[1] = bf16_bits_to_float(raw.x >> 16);
        z[2] = bf16_bits_to_float(raw.y & 0xffffu); z[3] = bf16_bits_to_float(raw.y >> 16);
    }
    if (!is_v && a.rope_style)
        warp_rope128(z, lane, a.rope_cos + (size_t)tok_pos(a, t) * 64, a.rope_sin + (size_t)tok_pos(a, t) * 64, a.rope_style);
    if (T.rotate) warp_fwht128(z, lane);
    if (T.has_mean) {  // remove the (dequantised) windowed channel mean, Sec. 4.2
        const int ps = tok_pos(a, t), w = ps / DQ_WINDOW_TOKENS;
        const size_t mi = ((size_t)tok_seq(a, t) * a.max_windows + w) * Hkv + h;
        uint32_t q4;
        float sc;
        if (a.mean_mode == DQ_MEAN_REUSE && ps % DQ_WINDOW_TOKENS == 0) {
            // first position of a window: carry the previous window's mean forward (window 0: zero).
            // Rows are per head, so this warp is the only writer and reader of the row in this call.
            q4 = 0u; sc = 0.f;
            if (w > 0) {
                const size_t src = mi - (size_t)Hkv;
                q4 = *reinterpret_cast<const uint32_t*>(a.mean_q + src * kN + 4 * lane);
                sc = a.mean_scale[src];
            }
            *reinterpret_cast<uint32_t*>(a.mean_q + mi * kN + 4 * lane) = q4;
            if (lane == 0) a.mean_scale[mi] = sc;
        } else {
            sc = a.mean_scale[mi];
            q4 = *reinterpret_cast<const uint32_t*>(a.mean_q + mi * kN + 4 * lane);
        }
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
        if (PAIR) drift_pair(T, z, s, o, sym); else drift(T, z, s, o, sym);
        // Refit: least squares of z on the symbols; binary64 sums in a fixed order
        double sa = (double)z[0], sb = __dmul_rn((double)sym[0], (double)z[0]);
        int sm = (int)sym[0], smm = (int)(sym[0] * sym[0]);
#pragma unroll
        for (int e = 1; e < 4; ++e) {
            sa = __dadd_rn(sa, (double)z[e]);
            sb = __dadd_rn(sb, __dmul_rn((double)sym[e], (double)z[e]));
            sm += (int)sym[e];
            smm += (int)(sym[e] * sym[e]);
        }
#pragma unroll
        for (int d = 16; d >= 1; d >>= 1) {
            sa = __dadd_rn(sa, __shfl_xor_sync(kFull, sa, d));
            sb = __dadd_rn(sb, __shfl_xor_sync(kFull, sb, d));
        }
        const long long Sm = __reduce_add_sync(kFull, sm), Smm = __reduce_add_sync(kFull, smm);
        const long long den = (long long)kN * Smm - Sm * Sm;
        double sd = (double)s, od = (double)o;
        if (den != 0) {
            sd = __ddiv_rn(__dsub_rn(__dmul_rn((double)kN, sb), __dmul_rn((double)Sm, sa)), (double)den);
            od = __ddiv_rn(__dsub_rn(sa, __dmul_rn(sd, (double)Sm)), (double)kN);
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
            const uint32_t len = PAIR ? drift_pair(T, z, sf, of, sym) : drift(T, z, sf, of, sym);   // second Drift, fp16 grid
            if (len > ((uint32_t)T.budget_bits << 16)) {
#pragma unroll
                for (int e = 0; e < 4; ++e) sym[e] = (T.central >> (8 * e)) & 0xffu;
                st_fallback = 1;
            }
        }
    }
    if (degenerate) {
        s16 = __ushort_as_half(0);
        o16 = __float2half_rn(mn);
#pragma unroll
        for (int e = 0; e < 4; ++e) sym[e] = (T.central >> (8 * e)) & 0xffu;
    }

    StreamQuantised r;
    r.hdr0 = (uint32_t)__half_as_ushort(s16) | ((uint32_t)__half_as_ushort(o16) << 16);
    r.flags = st_fallback | (degenerate ? 2u : 0u) | (st_refit << 2);
    r.sym = sym[0] | (sym[1] << 8) | (sym[2] << 16) | (sym[3] << 24);
    return r;
}

// One warp per stream (token, KV head); lane l owns elements 4l .. 4l+3.  blockIdx.y selects
// the tensor kind when keys and values are encoded by one launch.
// MINB CTAs per SM: 2 leaves every thread 128 registers (lowest latency: the single-token step), 4 trades a
// few spills for twice the resident warps (throughput: prefill, bulk encodes).
// WARPS streams per CTA: 8 normally; the decode step uses 16 (512 threads at full register budget) so that its
// 2 B Hkv streams occupy few SMs while the attention kernel runs on all the others.
template <int MINB, int WARPS, bool PAIR>
__global__ void __launch_bounds__(WARPS * 32, MINB)
dq_encode_kernel(const __grid_constant__ DqDevTable TK, const __grid_constant__ DqDevTable TV,
                 const __grid_constant__ DqPairEnc PK, const __grid_constant__ DqPairEnc PV, const DqEncodeArgs a) {
    __shared__ EncTable T;
    __shared__ uint8_t s_bytes[WARPS][DQ_MAX_REC_BYTES];
    __shared__ __align__(4) uint8_t s_sym[WARPS][kN];
    // Decode-step mode: the kernels after this one start while it runs and take their own launch as proof
    // that everything before this kernel has finished, so the trigger comes after the wait (and after the
    // hand-over words are cleared).  Otherwise: trigger first, so that the next kernel's launch overlaps this one.
    if (!a.step_flags) dqdev::pdl_launch_dependents();
    const bool is_v = a.do_k ? (blockIdx.y == 1) : true;
    load_enc_table(T, TK, TV, PK, PV, is_v);
    __syncthreads();
    dqdev::pdl_wait_prior_grid();   // inputs and the cache may be written / read by the previous kernel
    if (a.step_flags) {
        if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x < 4) {
            a.step_flags[threadIdx.x] = 0;
            __threadfence();
        }
        __syncthreads();
        dqdev::pdl_launch_dependents();
    }
    const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
    const long long wid = (long long)blockIdx.x * WARPS + wib;
    if (wid >= (long long)a.T * a.Hkv) return;
    if (tok_pos(a, (int)(wid / a.Hkv)) < 0) return;   // decode-step mode: an empty sequence has no new token
    const int t = (int)(wid / a.Hkv), h = (int)(wid % a.Hkv), Hkv = a.Hkv;
    uint8_t* cont = is_v ? a.v_cont : a.k_cont;

    const StreamQuantised sq = quantise_stream<PAIR>(T, a, is_v, t, h, lane);
    // rANS, Eq. (rans) Enc on symbols 127 .. 0 so that decoding runs forward.  Every lane
    // carries the same state (the symbols come from shared memory); lane 0 records the bytes.
    // (paired symbols: the lane's two pair indices u = a M + b; the coder then runs over 64 symbols)
    if (PAIR) {
        const uint32_t M = (uint32_t)T.M;
        const uint32_t u0 = (sq.sym & 0xffu) * M + ((sq.sym >> 8) & 0xffu), u1 = ((sq.sym >> 16) & 0xffu) * M + (sq.sym >> 24);
        *reinterpret_cast<uint16_t*>(&s_sym[wib][2 * lane]) = (uint16_t)(u0 | (u1 << 8));
    } else {
        *reinterpret_cast<uint32_t*>(&s_sym[wib][4 * lane]) = sq.sym;
    }
    __syncwarp();
    uint32_t xs = 1u << (T.sigma - 9);   // L: 2^23, or 2^15 with the 24-bit state
    int k = 0;
    // emitted bytes go to shared memory through stores the compiler does not treat as aliasing
    // the symbol / table loads, so those loads are issued ahead of the serial state chain
    const uint32_t bytes_addr = dqdev::smem_addr(s_bytes[wib]);
#pragma unroll 8
    for (int j = (PAIR ? kN / 2 : kN) - 1; j >= 0; --j) {
        const uint32_t m = s_sym[wib][j];
        const uint32_t rcp = T.rcp[m], rsh = T.rsh[m], bias = T.bias[m], cmpl = T.cmpl[m], thr = T.thr[m];
        if (xs >= thr) {  // at most once: xs < 2^8 L <= 2^8 * (f L)
            if (lane == 0) asm volatile("st.shared.u8 [%0], %1;" ::"r"(bytes_addr + k), "r"(xs & 0xffu));
            ++k;
            xs >>= 8;
        }
        xs = (__umulhi(xs, rcp) >> rsh) * cmpl + (xs + bias);
    }
    __syncwarp();
    asm volatile("" ::: "memory");
    const uint32_t hdr0 = sq.hdr0;
    const int sl = a.slot[t];
    uint8_t* rec = cont + (((size_t)(sl / DQ_PAGE_TOKENS) * Hkv + h) * DQ_PAGE_TOKENS +
                           (size_t)(sl % DQ_PAGE_TOKENS)) * T.rec;
    const int pay = 4 + (T.sigma >> 3);              // first payload byte: after (s, o) and the final state
    const int used = min(pay + k, T.rec);            // the budget test keeps pay + k <= rec
    for (int i = lane; i < T.rec; i += 32) {
        uint8_t v = 0;
        if (i < 4) v = (uint8_t)(hdr0 >> (8 * i));
        else if (i < pay) v = (uint8_t)(xs >> (8 * (i - 4)));
        else if (i < used) v = s_bytes[wib][k - 1 - (i - pay)];
        rec[i] = v;
    }
    if (a.status && lane == 0) {
        if (sq.flags & 1u) atomicAdd(a.status + 0, 1u);
        if (sq.flags & 2u) atomicAdd(a.status + 1, 1u);
        if (sq.flags & 4u) atomicAdd(a.status + 2, 1u);
        atomicMax(a.status + 3, (uint32_t)(pay + k));
    }
}


// Throughput variant for calls with many streams: a CTA of 4 warps takes 32 consecutive streams.
// Each warp quantises 8 of them (steps 1-6 of Algorithm 1, as above) and leaves the symbols in
// shared memory; then ONE warp entropy-codes all 32 streams at once, lane = stream, so the serial
// rANS chain costs one instruction stream per 32 streams instead of one per stream with 32
// redundant lanes.  Symbols are stored [position][stream] and emitted bytes [byte index][stream] so
// that the lanes of that warp touch consecutive bytes.  Small CTAs, 8 per SM at 64 registers: the
// other warps of a CTA idle during its rANS pass, so that pass should be a small part of a small CTA.
#ifndef DQ_B32_MINB
#define DQ_B32_MINB 8
#endif
#ifndef DQ_B32_WARPS
#define DQ_B32_WARPS 4
#endif
constexpr int kB32 = 32;                 // streams per CTA
constexpr int kB32SymStride = 36;        // bytes per position row (32 streams + pad against bank conflicts)
constexpr int kB32Warps = DQ_B32_WARPS;
constexpr int kB32PairMinBlocks = 4;   // paired symbols: the pair search wants 128 registers (7.9 ms against 12.5 ms at 8 CTAs per SM, config 2 prefill)
template <int MINB, bool PAIR>
__global__ void __launch_bounds__(kB32Warps * 32, MINB)
dq_encode_batch32_kernel(const __grid_constant__ DqDevTable TK, const __grid_constant__ DqDevTable TV,
                         const __grid_constant__ DqPairEnc PK, const __grid_constant__ DqPairEnc PV, const DqEncodeArgs a) {
    __shared__ EncTable T;
    __shared__ __align__(4) uint8_t s_symT[kN * kB32SymStride];
    __shared__ uint8_t s_bytesT[DQ_MAX_REC_BYTES * kB32];
    __shared__ uint32_t s_hdr[kB32], s_xs[kB32], s_k[kB32];
    __shared__ unsigned long long s_rec[kB32];   // record addresses
    dqdev::pdl_launch_dependents();
    const bool is_v = a.do_k ? (blockIdx.y == 1) : true;
    load_enc_table(T, TK, TV, PK, PV, is_v);
    __syncthreads();
    dqdev::pdl_wait_prior_grid();
    const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
    const long long total = (long long)a.T * a.Hkv;
    const long long first = (long long)blockIdx.x * kB32;
    const int ns = (int)min((long long)kB32, total - first);
    uint8_t* cont = is_v ? a.v_cont : a.k_cont;

    for (int i = wib; i < ns; i += kB32Warps) {   // quantise: warp w takes streams w, w + warps, ...
        const long long wid = first + i;
        const int t = (int)(wid / a.Hkv), h = (int)(wid % a.Hkv);
        const StreamQuantised sq = quantise_stream<PAIR>(T, a, is_v, t, h, lane);
        if (PAIR) {   // the lane's two pair indices u = a M + b at positions 2 lane, 2 lane + 1
            const uint32_t M = (uint32_t)T.M;
            s_symT[(2 * lane) * kB32SymStride + i] = (uint8_t)((sq.sym & 0xffu) * M + ((sq.sym >> 8) & 0xffu));
            s_symT[(2 * lane + 1) * kB32SymStride + i] = (uint8_t)(((sq.sym >> 16) & 0xffu) * M + (sq.sym >> 24));
        } else {
#pragma unroll
            for (int e = 0; e < 4; ++e) s_symT[(4 * lane + e) * kB32SymStride + i] = (uint8_t)(sq.sym >> (8 * e));
        }
        if (lane == 0) {
            s_hdr[i] = sq.hdr0;
            const int sl = a.slot[t];
            s_rec[i] = (unsigned long long)(cont + (((size_t)(sl / DQ_PAGE_TOKENS) * a.Hkv + h) * DQ_PAGE_TOKENS +
                                                    (size_t)(sl % DQ_PAGE_TOKENS)) * T.rec);
            if (a.status) {
                if (sq.flags & 1u) atomicAdd(a.status + 0, 1u);
                if (sq.flags & 2u) atomicAdd(a.status + 1, 1u);
                if (sq.flags & 4u) atomicAdd(a.status + 2, 1u);
            }
        }
    }
    __syncthreads();
    if (wib == 0 && lane < ns) {   // rANS, Eq. (rans) Enc on symbols 127 .. 0; lane = stream
        uint32_t xs = 1u << (T.sigma - 9), k = 0;
#pragma unroll 4
        for (int j = (PAIR ? kN / 2 : kN) - 1; j >= 0; --j) {
            const uint32_t m = s_symT[j * kB32SymStride + lane];
            const uint32_t rcp = T.rcp[m], rsh = T.rsh[m], bias = T.bias[m], cmpl = T.cmpl[m], thr = T.thr[m];
            if (xs >= thr) {   // at most once: xs < 2^8 L <= 2^8 * (f L)
                if (k < DQ_MAX_REC_BYTES) s_bytesT[k * kB32 + lane] = (uint8_t)xs;   // the budget test keeps k < rec - 8
                ++k;
                xs >>= 8;
            }
            xs = (__umulhi(xs, rcp) >> rsh) * cmpl + (xs + bias);
        }
        s_xs[lane] = xs;
        s_k[lane] = k;
        if (a.status) atomicMax(a.status + 3, 4u + (uint32_t)(T.sigma >> 3) + k);
    }
    __syncthreads();
    const int rec = T.rec, pay = 4 + (T.sigma >> 3);
    for (int idx = threadIdx.x; idx < ns * rec; idx += blockDim.x) {   // records out: header, state, k bytes, then zeros
        const int si = idx / rec, i = idx - si * rec;
        const int k = (int)s_k[si], used = min(pay + k, rec);
        uint8_t v = 0;
        if (i < 4) v = (uint8_t)(s_hdr[si] >> (8 * i));
        else if (i < pay) v = (uint8_t)(s_xs[si] >> (8 * (i - 4)));
        else if (i < used) v = s_bytesT[(k - 1 - (i - pay)) * kB32 + si];   // emitted last = read first
        reinterpret_cast<uint8_t*>(s_rec[si])[i] = v;
    }
}

// rANS encode of one stream by one warp (Eq. rans Enc on symbols n-1 .. 0 so that decoding runs
// forward).  Every lane carries the same state; lane 0 records the emitted bytes (in emission
// order) at `bytes_addr` in shared memory.  The per-symbol table entries do not depend on the
// state, so they are fetched four symbols ahead of the serial state chain.
//   ent[m] = {rcp, bias | (256 - f) << 10 | rsh << 19}
__device__ __forceinline__ void rans_encode_warp(const uint2* ent, const uint8_t* sym, int n, uint32_t bytes_addr,
                                                 int cap, int lane, uint32_t& xs_out, int& k_out) {
    uint32_t xs = kL;
    int k = 0;
    const uint32_t* sym4 = reinterpret_cast<const uint32_t*>(sym);
    uint2 cur[4], nxt[4];
    {
        const uint32_t m4 = sym4[n / 4 - 1];
#pragma unroll
        for (int i = 0; i < 4; ++i) nxt[i] = ent[(m4 >> (8 * i)) & 255u];
    }
#pragma unroll 1
    for (int j4 = n / 4 - 1; j4 >= 0; --j4) {
#pragma unroll
        for (int i = 0; i < 4; ++i) cur[i] = nxt[i];
        if (j4 > 0) {
            const uint32_t m4 = sym4[j4 - 1];
#pragma unroll
            for (int i = 0; i < 4; ++i) nxt[i] = ent[(m4 >> (8 * i)) & 255u];
        }
#pragma unroll
        for (int i = 3; i >= 0; --i) {
            const uint32_t aux = cur[i].y, cmpl = (aux >> 10) & 511u;
            const bool emit = xs >= ((256u - cmpl) << 23);   // at most once: xs < 2^31 <= 2^8 * (f << 23)
            if (emit && lane == 0 && k < cap) asm volatile("st.shared.u8 [%0], %1;" ::"r"(bytes_addr + k), "r"(xs & 0xffu));
            k += emit ? 1 : 0;
            xs = emit ? (xs >> 8) : xs;
            xs = (__umulhi(xs, cur[i].x) >> (aux >> 19)) * cmpl + (xs + (aux & 1023u));
        }
    }
    xs_out = xs;
    k_out = k;
}

// ------------------------------------------------------- token-wide streams (hs heads)

// Cross-warp pieces of a stream that spans hs heads: one CTA per stream, warp w holds head w
// (4 values per lane, as above).  Reductions over the stream go warp -> shared slot -> CTA
// barrier; slots are double-buffered by call parity so one barrier per reduction suffices.
struct WideShared {
    float fmax[2][DQ_MAX_STREAM_HEADS], fmin[2][DQ_MAX_STREAM_HEADS];
    uint32_t len[2][DQ_MAX_STREAM_HEADS];
    double sa[DQ_MAX_STREAM_HEADS], sb[DQ_MAX_STREAM_HEADS];
    int sm[DQ_MAX_STREAM_HEADS], smm[DQ_MAX_STREAM_HEADS];
    uint2 ent[DQ_MAX_PAIRS];    // rANS encode entries {rcp, bias | (256 - f) << 10 | rsh << 19} (levels, or pairs u = a M + b)
};

// Function Drift of Algorithm 1 for a stream held by hs warps; same arithmetic as drift_m, with
// the extrema of D and the code length taken over the whole stream.
template <int M>
__device__ __noinline__ uint32_t drift_wide_m(const EncTable& T, WideShared& W, int hs, int wib, uint32_t& parity,
                                              float z0, float z1, float z2, float z3, float s, float o,
                                              uint32_t& sym_packed) {
    const float z[4] = {z0, z1, z2, z3};
    const int lane = threadIdx.x & 31;
    float tm[M], rm[M];
    uint32_t Km[M];   // ceil(65536 r_m) << 8 | m: the minimum tree carries one word for length and index
#pragma unroll
    for (int m = 0; m < M; ++m) {
        tm[m] = __fmaf_rn((float)m, s, o);
        rm[m] = T.r[m];
        Km[m] = (T.R[m] << 8) | (uint32_t)m;
    }
    float D[4][M];
    float maxD = -INFINITY, minD = INFINITY;
#pragma unroll
    for (int e = 0; e < 4; ++e)
#pragma unroll
        for (int m = 0; m < M; ++m) {
            const float d = __fsub_rn(z[e], tm[m]);
            D[e][m] = __fmul_rn(d, d);
            maxD = fmaxf(maxD, D[e][m]);
            minD = fminf(minD, D[e][m]);
        }
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) {
        maxD = fmaxf(maxD, __shfl_xor_sync(kFull, maxD, d));
        minD = fminf(minD, __shfl_xor_sync(kFull, minD, d));
    }
    if (lane == 0) { W.fmax[parity][wib] = maxD; W.fmin[parity][wib] = minD; }
    __syncthreads();
    for (int w = 0; w < hs; ++w) { maxD = fmaxf(maxD, W.fmax[parity][w]); minD = fminf(minD, W.fmin[parity][w]); }
    parity ^= 1u;
    const uint32_t budget = (uint32_t)T.budget_bits << 16;
    float lam_hi = __fmul_rn(8.0f, __fsub_rn(maxD, minD));
    float lam_lo = __fmul_rn(lam_hi, 0x1p-40f);
    uint32_t len = 0, sym[4] = {0u, 0u, 0u, 0u};
    // Early-exit variant: when each of the 12 tests passes, the upper end walks hi <- sqrt(lo hi) twelve
    // times with lo fixed; sweep -1 evaluates that multiplier and ends the search if its assignment fits.
    float lam_e = lam_hi;
    if (T.early_exit)
        for (int i = 0; i < 12; ++i) lam_e = __fsqrt_rn(__fmul_rn(lam_lo, lam_e));
#pragma unroll 1
    for (int it = T.early_exit ? -1 : 0; it <= 12; ++it) {
        const float lam = (it < 0) ? lam_e : (it < 12) ? __fsqrt_rn(__fmul_rn(lam_lo, lam_hi)) : lam_hi;
        uint32_t cost_sum = 0;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            float c[M];
            uint32_t key[M];
#pragma unroll
            for (int m = 0; m < M; ++m) { c[m] = __fmaf_rn(lam, rm[m], D[e][m]); key[m] = Km[m]; }
#pragma unroll
            for (int w = 1; w < M; w <<= 1)
#pragma unroll
                for (int m = 0; m + w < M; m += 2 * w)
                    if (c[m + w] < c[m]) { c[m] = c[m + w]; key[m] = key[m + w]; }
            sym[e] = key[0];
            cost_sum += key[0];
        }
        const uint32_t wl = __reduce_add_sync(kFull, cost_sum >> 8);
        if (lane == 0) W.len[parity][wib] = wl;
        __syncthreads();
        len = 0;
        for (int w = 0; w < hs; ++w) len += W.len[parity][w];
        parity ^= 1u;
        if (it < 0) {
            if (len <= budget) break;   // uniform across the CTA: every warp sees the same stream-wide length
        } else if (it < 12) {
            if (len <= budget) lam_hi = lam; else lam_lo = lam;
        }
    }
    sym_packed = (sym[0] & 0xffu) | ((sym[1] & 0xffu) << 8) | ((sym[2] & 0xffu) << 16) | (sym[3] << 24);
    return len;
}

__device__ __forceinline__ uint32_t drift_wide(const EncTable& T, WideShared& W, int hs, int wib, uint32_t& parity,
                                               const float (&z)[4], float s, float o, uint32_t (&sym)[4]) {
    uint32_t packed = 0, len = 0;
    switch (T.M) {   // uniform across the CTA
#define DQ_DRIFT_CASE(M_) case M_: len = drift_wide_m<M_>(T, W, hs, wib, parity, z[0], z[1], z[2], z[3], s, o, packed); break;
        DQ_DRIFT_CASE(2) DQ_DRIFT_CASE(3) DQ_DRIFT_CASE(4) DQ_DRIFT_CASE(5) DQ_DRIFT_CASE(6) DQ_DRIFT_CASE(7)
        DQ_DRIFT_CASE(8) DQ_DRIFT_CASE(9) DQ_DRIFT_CASE(10) DQ_DRIFT_CASE(11) DQ_DRIFT_CASE(12) DQ_DRIFT_CASE(13)
        DQ_DRIFT_CASE(14) DQ_DRIFT_CASE(15) DQ_DRIFT_CASE(16)
#undef DQ_DRIFT_CASE
        default: break;
    }
#pragma unroll
    for (int e = 0; e < 4; ++e) sym[e] = (packed >> (8 * e)) & 0xffu;
    return len;
}

// Drift for paired symbols on a stream held by hs warps: the pair search of drift_pair_m with the extrema of D
// and the code length taken over the whole stream, as in drift_wide_m.
template <int M>
__device__ __noinline__ uint32_t drift_wide_pair_m(const EncTable& T, WideShared& W, int hs, int wib, uint32_t& parity,
                                                   float z0, float z1, float z2, float z3, float s, float o,
                                                   uint32_t& sym_packed) {
    const float z[4] = {z0, z1, z2, z3};
    const int lane = threadIdx.x & 31;
    float D[4][M];
    float maxD = -INFINITY, minD = INFINITY;
#pragma unroll
    for (int m = 0; m < M; ++m) {
        const float tm = __fmaf_rn((float)m, s, o);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float d = __fsub_rn(z[e], tm);
            D[e][m] = __fmul_rn(d, d);
            maxD = fmaxf(maxD, D[e][m]);
            minD = fminf(minD, D[e][m]);
        }
    }
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) {
        maxD = fmaxf(maxD, __shfl_xor_sync(kFull, maxD, d));
        minD = fminf(minD, __shfl_xor_sync(kFull, minD, d));
    }
    if (lane == 0) { W.fmax[parity][wib] = maxD; W.fmin[parity][wib] = minD; }
    __syncthreads();
    for (int w = 0; w < hs; ++w) { maxD = fmaxf(maxD, W.fmax[parity][w]); minD = fminf(minD, W.fmin[parity][w]); }
    parity ^= 1u;
    const uint32_t budget = (uint32_t)T.budget_bits << 16;
    float lam_hi = __fmul_rn(16.0f, __fsub_rn(maxD, minD));
    float lam_lo = __fmul_rn(lam_hi, 0x1p-40f);
    uint32_t len = 0, psym[2] = {0u, 0u};
    float lam_e = lam_hi;
    if (T.early_exit)
        for (int i = 0; i < 12; ++i) lam_e = __fsqrt_rn(__fmul_rn(lam_lo, lam_e));
#pragma unroll 1
    for (int it = T.early_exit ? -1 : 0; it <= 12; ++it) {
        const float lam = (it < 0) ? lam_e : (it < 12) ? __fsqrt_rn(__fmul_rn(lam_lo, lam_hi)) : lam_hi;
        uint32_t cost_sum = 0;
#pragma unroll
        for (int p = 0; p < 2; ++p) {
            float best = 0.f;
            uint32_t bkey = 0u;
#pragma unroll
            for (int a = 0; a < M; ++a) {
                float c[M];
                uint32_t key[M];
#pragma unroll
                for (int b = 0; b < M; ++b) {
                    const uint2 e = T.prk[a * M + b];
                    c[b] = __fmaf_rn(lam, __uint_as_float(e.x), __fadd_rn(D[2 * p][a], D[2 * p + 1][b]));
                    key[b] = e.y;
                }
#pragma unroll
                for (int w = 1; w < M; w <<= 1)
#pragma unroll
                    for (int b = 0; b + w < M; b += 2 * w)
                        if (c[b + w] < c[b]) { c[b] = c[b + w]; key[b] = key[b + w]; }
                if (a == 0 || c[0] < best) { best = c[0]; bkey = key[0]; }   // an earlier row keeps equal costs
            }
            psym[p] = bkey;
            cost_sum += bkey;
        }
        const uint32_t wl = __reduce_add_sync(kFull, cost_sum >> 8);
        if (lane == 0) W.len[parity][wib] = wl;
        __syncthreads();
        len = 0;
        for (int w = 0; w < hs; ++w) len += W.len[parity][w];
        parity ^= 1u;
        if (it < 0) {
            if (len <= budget) break;   // uniform across the CTA
        } else if (it < 12) {
            if (len <= budget) lam_hi = lam; else lam_lo = lam;
        }
    }
    const uint32_t u0 = psym[0] & 0xffu, u1 = psym[1] & 0xffu;
    sym_packed = (u0 / M) | ((u0 % M) << 8) | ((u1 / M) << 16) | ((u1 % M) << 24);
    return len;
}

__device__ __forceinline__ uint32_t drift_wide_pair(const EncTable& T, WideShared& W, int hs, int wib, uint32_t& parity,
                                                    const float (&z)[4], float s, float o, uint32_t (&sym)[4]) {
    uint32_t packed = 0, len = 0;
    switch (T.M) {   // uniform across the CTA
#define DQ_DRIFT_CASE(M_) case M_: len = drift_wide_pair_m<M_>(T, W, hs, wib, parity, z[0], z[1], z[2], z[3], s, o, packed); break;
        DQ_DRIFT_CASE(2) DQ_DRIFT_CASE(3) DQ_DRIFT_CASE(4) DQ_DRIFT_CASE(5) DQ_DRIFT_CASE(6) DQ_DRIFT_CASE(7)
        DQ_DRIFT_CASE(8) DQ_DRIFT_CASE(9)
#undef DQ_DRIFT_CASE
        default: break;
    }
#pragma unroll
    for (int e = 0; e < 4; ++e) sym[e] = (packed >> (8 * e)) & 0xffu;
    return len;
}

// Table fields of one tensor kind into shared memory (threads 0 .. DQ_MAX_PAIRS - 1 of 3 rounds of 32 + thread 0;
// a CTA has at least 64 threads).
__device__ __forceinline__ void load_wide_table(EncTable& T, WideShared& W, const DqDevTable& TK, const DqDevTable& TV,
                                                const DqPairEnc& PK, const DqPairEnc& PV, bool is_v) {
    const int pair = is_v ? TV.pair : TK.pair;
    if (threadIdx.x < DQ_MAX_LEVELS) {
        const int i = threadIdx.x;
        T.r[i] = is_v ? TV.r[i] : TK.r[i];
        T.R[i] = is_v ? TV.R[i] : TK.R[i];
        if (!pair) W.ent[i] = make_uint2(is_v ? TV.enc_rcp[i] : TK.enc_rcp[i], is_v ? TV.enc_aux[i] : TK.enc_aux[i]);
    }
    if (pair)
        for (int i = threadIdx.x; i < DQ_MAX_PAIRS; i += blockDim.x) {
            W.ent[i] = make_uint2(is_v ? PV.enc_rcp[i] : PK.enc_rcp[i], is_v ? PV.enc_aux[i] : PK.enc_aux[i]);
            T.prk[i] = make_uint2(__float_as_uint(is_v ? PV.r[i] : PK.r[i]), ((is_v ? PV.R[i] : PK.R[i]) << 8) | (uint32_t)i);
        }
    if (threadIdx.x == 0) {
        T.M = is_v ? TV.M : TK.M; T.rec = is_v ? TV.rec : TK.rec; T.mstar = is_v ? TV.mstar : TK.mstar;
        T.budget_bits = is_v ? TV.budget_bits : TK.budget_bits;
        T.has_mean = is_v ? TV.has_mean : TK.has_mean; T.rotate = is_v ? TV.rotate : TK.rotate;
        T.early_exit = is_v ? TV.early_exit : TK.early_exit; T.sigma = 32;   // token-wide streams keep the 32-bit state
        T.pair = pair;
        const uint32_t ms = (uint32_t)T.mstar, us = (uint32_t)(is_v ? TV.ustar : TK.ustar), M = (uint32_t)T.M;
        T.central = pair ? (us / M) * 0x00010001u + (us % M) * 0x01000100u : ms * 0x01010101u;
    }
}

struct WideQuantised {
    uint32_t hdr0;      // s fp16 | o fp16 << 16
    uint32_t flags;     // 1: all-central fallback, 2: constant stream, 4: refit rejected
};

// Steps 1-6 of Algorithm 1 for the stream (token t, group grp) held by the CTA's hs warps
// (warp w owns head grp * hs + w, lane l its elements 4l .. 4l+3 = stream positions
// 128 w + 4 l + e): rotation, mean removal, min-max grid, drift, refit, fp16 metadata, second
// drift.  The final symbols go to s_sym (visible to the whole CTA on return).
// PAIR: rANS symbols are pairs of levels; s_sym then receives the pair index u = a M + b of the values
// (2i, 2i + 1) at symbol position i (n / 2 positions).
template <bool PAIR>
__device__ __forceinline__ WideQuantised wide_quantise(const EncTable& T, WideShared& W, const DqEncodeArgs& a,
                                                       bool is_v, int t, int grp, uint8_t* s_sym, int sym_stride,
                                                       uint32_t& parity) {
    const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
    const int hs = blockDim.x >> 5, Hkv = a.Hkv, h = grp * hs + wib;
    const int n = hs * kN;
    const uint16_t* x = static_cast<const uint16_t*>(is_v ? a.v_bf16 : a.k_bf16);
    float z[4];
    {
        const uint2 raw = *reinterpret_cast<const uint2*>(x + ((size_t)t * Hkv + h) * kN + 4 * lane);
        z[0] = bf16_bits_to_float(raw.x & 0xffffu); z[1] = bf16_bits_to_float(raw.x >> 16);
        z[2] = bf16_bits_to_float(raw.y & 0xffffu); z[3] = bf16_bits_to_float(raw.y >> 16);
    }
    if (!is_v && a.rope_style)
        warp_rope128(z, lane, a.rope_cos + (size_t)a.pos[t] * 64, a.rope_sin + (size_t)a.pos[t] * 64, a.rope_style);
    if (T.rotate) warp_fwht128(z, lane);
    if (T.has_mean) {  // remove the (dequantised) windowed channel mean of this head, Sec. 4.2
        const int ps = a.pos[t], w = ps / DQ_WINDOW_TOKENS;
        const size_t mi = ((size_t)a.seq_id[t] * a.max_windows + w) * Hkv + h;
        uint32_t q4;
        float sc;
        if (a.mean_mode == DQ_MEAN_REUSE && ps % DQ_WINDOW_TOKENS == 0) {
            q4 = 0u; sc = 0.f;   // first position of a window: carry the previous window's mean forward
            if (w > 0) {
                const size_t src = mi - (size_t)Hkv;
                q4 = *reinterpret_cast<const uint32_t*>(a.mean_q + src * kN + 4 * lane);
                sc = a.mean_scale[src];
            }
            *reinterpret_cast<uint32_t*>(a.mean_q + mi * kN + 4 * lane) = q4;
            if (lane == 0) a.mean_scale[mi] = sc;
        } else {
            sc = a.mean_scale[mi];
            q4 = *reinterpret_cast<const uint32_t*>(a.mean_q + mi * kN + 4 * lane);
        }
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
    if (lane == 0) { W.fmax[parity][wib] = mx; W.fmin[parity][wib] = mn; }
    __syncthreads();
    for (int w = 0; w < hs; ++w) { mx = fmaxf(mx, W.fmax[parity][w]); mn = fminf(mn, W.fmin[parity][w]); }
    parity ^= 1u;

    uint32_t sym[4];
    __half s16 = __ushort_as_half(0), o16 = __ushort_as_half(0);
    bool degenerate = !(mx > mn);
    uint32_t flags = 0;
    if (!degenerate) {   // uniform across the CTA: mx and mn are stream-wide
        const float o = mn;                                         // FitMinMax, Eq. (affine_token)
        const float s = __fdiv_rn(__fsub_rn(mx, mn), (float)(T.M - 1));
        if (PAIR) drift_wide_pair(T, W, hs, wib, parity, z, s, o, sym); else drift_wide(T, W, hs, wib, parity, z, s, o, sym);
        // Refit: head sums as in the per-head encoder (lane order, then xor butterfly), added in head order
        double sa = (double)z[0], sb = __dmul_rn((double)sym[0], (double)z[0]);
        int sm = (int)sym[0], smm = (int)(sym[0] * sym[0]);
#pragma unroll
        for (int e = 1; e < 4; ++e) {
            sa = __dadd_rn(sa, (double)z[e]);
            sb = __dadd_rn(sb, __dmul_rn((double)sym[e], (double)z[e]));
            sm += (int)sym[e];
            smm += (int)(sym[e] * sym[e]);
        }
#pragma unroll
        for (int d = 16; d >= 1; d >>= 1) {
            sa = __dadd_rn(sa, __shfl_xor_sync(kFull, sa, d));
            sb = __dadd_rn(sb, __shfl_xor_sync(kFull, sb, d));
        }
        sm = __reduce_add_sync(kFull, sm);
        smm = __reduce_add_sync(kFull, smm);
        __syncthreads();   // the previous stream's readers of W.sa .. are done
        if (lane == 0) { W.sa[wib] = sa; W.sb[wib] = sb; W.sm[wib] = sm; W.smm[wib] = smm; }
        __syncthreads();
        sa = W.sa[0]; sb = W.sb[0];
        long long Sm = W.sm[0], Smm = W.smm[0];
        for (int w = 1; w < hs; ++w) {
            sa = __dadd_rn(sa, W.sa[w]);
            sb = __dadd_rn(sb, W.sb[w]);
            Sm += W.sm[w]; Smm += W.smm[w];
        }
        const long long den = (long long)n * Smm - Sm * Sm;
        double sd = (double)s, od = (double)o;
        if (den != 0) {
            sd = __ddiv_rn(__dsub_rn(__dmul_rn((double)n, sb), __dmul_rn((double)Sm, sa)), (double)den);
            od = __ddiv_rn(__dsub_rn(sa, __dmul_rn(sd, (double)Sm)), (double)n);
        }
        s16 = __double2half(sd);                                    // fp16 metadata
        o16 = __double2half(od);
        float sf = __half2float(s16), of = __half2float(o16);
        if (!(isfinite(sf) && sf > 0.0f && isfinite(of))) {
            s16 = __float2half_rn(s);
            o16 = __float2half_rn(o);
            sf = __half2float(s16); of = __half2float(o16);
            flags |= 4u;
        }
        if (!(sf > 0.0f)) degenerate = true;
        else {
            const uint32_t len = PAIR ? drift_wide_pair(T, W, hs, wib, parity, z, sf, of, sym)
                                      : drift_wide(T, W, hs, wib, parity, z, sf, of, sym);   // second Drift, fp16 grid
            if (len > ((uint32_t)T.budget_bits << 16)) {
#pragma unroll
                for (int e = 0; e < 4; ++e) sym[e] = (T.central >> (8 * e)) & 0xffu;
                flags |= 1u;
            }
        }
    }
    if (degenerate) {
        s16 = __ushort_as_half(0);
        o16 = __float2half_rn(mn);
#pragma unroll
        for (int e = 0; e < 4; ++e) sym[e] = (T.central >> (8 * e)) & 0xffu;
        flags |= 2u;
    }
    // symbol of stream position j goes to s_sym[j * sym_stride]
    if (PAIR) {
        const uint32_t M = (uint32_t)T.M;
        s_sym[(wib * (kN / 2) + 2 * lane) * sym_stride] = (uint8_t)(sym[0] * M + sym[1]);
        s_sym[(wib * (kN / 2) + 2 * lane + 1) * sym_stride] = (uint8_t)(sym[2] * M + sym[3]);
    } else {
#pragma unroll
        for (int e = 0; e < 4; ++e) s_sym[(wib * kN + 4 * lane + e) * sym_stride] = (uint8_t)sym[e];
    }
    __syncthreads();
    WideQuantised r;
    r.hdr0 = (uint32_t)__half_as_ushort(s16) | ((uint32_t)__half_as_ushort(o16) << 16);
    r.flags = flags;
    return r;
}

// Record of one stream into the word-interleaved page layout (all threads of the CTA).
__device__ __forceinline__ void write_wide_record(uint8_t* cont, int groups, int grp, int rec, int slot, uint32_t hdr0,
                                                  uint32_t xs, int k, const uint8_t* bytes) {
    const int rec_words = (rec + 3) >> 2;
    uint8_t* blk = cont + ((size_t)(slot / DQ_PAGE_TOKENS) * groups + grp) * ((size_t)rec_words * 64) +
                   (size_t)(slot % DQ_PAGE_TOKENS) * 4;
    const int used = min(8 + k, rec);   // the budget test keeps 8 + k <= rec
    for (int i = threadIdx.x; i < rec_words * 4; i += blockDim.x) {
        uint8_t v = 0;
        if (i < 4) v = (uint8_t)(hdr0 >> (8 * i));
        else if (i < 8) v = (uint8_t)(xs >> (8 * (i - 4)));
        else if (i < used) v = bytes[k - 1 - (i - 8)];   // emitted last = read first
        blk[(size_t)(i >> 2) * 64 + (i & 3)] = v;
    }
}

__device__ __forceinline__ void add_status(uint32_t* status, uint32_t flags, int k) {
    if (!status) return;
    if (flags & 1u) atomicAdd(status + 0, 1u);
    if (flags & 2u) atomicAdd(status + 1, 1u);
    if (flags & 4u) atomicAdd(status + 2, 1u);
    atomicMax(status + 3, (uint32_t)(8 + k));
}

// One CTA of hs warps per stream (token, group of hs KV heads): lowest latency, used when a
// call holds few streams (a decode step).  blockIdx.y selects the tensor kind.
template <bool PAIR>
__global__ void __launch_bounds__(DQ_MAX_STREAM_HEADS * 32)
dq_encode_wide_kernel(const __grid_constant__ DqDevTable TK, const __grid_constant__ DqDevTable TV,
                      const __grid_constant__ DqPairEnc PK, const __grid_constant__ DqPairEnc PV, const DqEncodeArgs a) {
    __shared__ EncTable T;
    __shared__ __align__(16) WideShared W;
    __shared__ uint8_t s_bytes[DQ_MAX_WIDE_REC_BYTES];
    __shared__ __align__(4) uint8_t s_sym[DQ_MAX_STREAM_HEADS * kN];
    __shared__ uint32_t s_final[2];   // final state, bytes emitted
    dqdev::pdl_launch_dependents();
    const bool is_v = a.do_k ? (blockIdx.y == 1) : true;
    load_wide_table(T, W, TK, TV, PK, PV, is_v);
    __syncthreads();
    dqdev::pdl_wait_prior_grid();
    const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
    const int hs = blockDim.x >> 5, groups = a.Hkv / hs;
    const int t = (int)(blockIdx.x / groups), grp = (int)(blockIdx.x % groups);
    uint32_t parity = 0;
    const WideQuantised q = wide_quantise<PAIR>(T, W, a, is_v, t, grp, s_sym, 1, parity);
    if (wib == 0) {
        uint32_t xs;
        int k;
        rans_encode_warp(W.ent, s_sym, PAIR ? hs * (kN / 2) : hs * kN, dqdev::smem_addr(s_bytes), DQ_MAX_WIDE_REC_BYTES, lane, xs, k);
        if (lane == 0) { s_final[0] = xs; s_final[1] = (uint32_t)k; }
    }
    __syncthreads();
    asm volatile("" ::: "memory");
    write_wide_record(is_v ? a.v_cont : a.k_cont, groups, grp, T.rec, a.slot[t], q.hdr0, s_final[0], (int)s_final[1], s_bytes);
    if (threadIdx.x == 0) add_status(a.status, q.flags, (int)s_final[1]);
}

// Throughput variant for calls with many streams (prefill, a window's bulk encode): a CTA takes
// 32 consecutive streams; its hs warps quantise them one after the other, then one warp
// entropy-codes all 32 at once, lane = stream (symbols stored [position][stream], emitted bytes
// [byte index][stream]), so the serial rANS chain is paid once per 32 streams.
constexpr int kWB = 32;              // streams per CTA
constexpr int kWBSymStride = 36;     // bytes per position row
__host__ __device__ inline int wide_batch_smem(int hs, int rec) { return hs * kN * kWBSymStride + ((rec + 3) & ~3) * kWB; }

#ifndef DQ_ENCW_MINB
#define DQ_ENCW_MINB 3
#endif
template <bool PAIR>
__global__ void __launch_bounds__(DQ_MAX_STREAM_HEADS * 32, PAIR ? 2 : DQ_ENCW_MINB)
dq_encode_wide_batch_kernel(const __grid_constant__ DqDevTable TK, const __grid_constant__ DqDevTable TV,
                            const __grid_constant__ DqPairEnc PK, const __grid_constant__ DqPairEnc PV, const DqEncodeArgs a) {
    extern __shared__ __align__(16) uint8_t dyn[];
    __shared__ EncTable T;
    __shared__ __align__(16) WideShared W;
    __shared__ uint32_t s_hdr[kWB], s_flags[kWB], s_xs[kWB], s_k[kWB];
    dqdev::pdl_launch_dependents();
    const bool is_v = a.do_k ? (blockIdx.y == 1) : true;
    load_wide_table(T, W, TK, TV, PK, PV, is_v);
    __syncthreads();
    dqdev::pdl_wait_prior_grid();
    const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
    const int hs = blockDim.x >> 5, groups = a.Hkv / hs, n = hs * kN;
    uint8_t* s_symT = dyn;                                   // [n][kWBSymStride]
    uint8_t* s_bytesT = dyn + n * kWBSymStride;              // [rec][kWB]
    const int cap = (T.rec + 3) & ~3;
    const long long total = (long long)a.T * groups;
    const long long first = (long long)blockIdx.x * kWB;
    const int ns = (int)min((long long)kWB, total - first);
    uint32_t parity = 0;
    for (int i = 0; i < ns; ++i) {
        const long long sid = first + i;
        const WideQuantised q = wide_quantise<PAIR>(T, W, a, is_v, (int)(sid / groups), (int)(sid % groups), s_symT + i,
                                              kWBSymStride, parity);
        if (threadIdx.x == 0) { s_hdr[i] = q.hdr0; s_flags[i] = q.flags; }
    }
    if (wib == 0 && lane < ns) {   // rANS, Eq. (rans) Enc on symbols n-1 .. 0; lane = stream
        uint32_t xs = kL, k = 0;
#pragma unroll 4
        for (int j = (PAIR ? n / 2 : n) - 1; j >= 0; --j) {
            const uint32_t m = s_symT[j * kWBSymStride + lane];
            const uint2 e = W.ent[m];
            const uint32_t cmpl = (e.y >> 10) & 511u;
            if (xs >= ((256u - cmpl) << 23)) {   // at most once: xs < 2^31 <= 2^8 * (f << 23)
                if ((int)k < cap) s_bytesT[k * kWB + lane] = (uint8_t)xs;   // the budget test keeps k < rec - 8
                ++k;
                xs >>= 8;
            }
            xs = (__umulhi(xs, e.x) >> (e.y >> 19)) * cmpl + (xs + (e.y & 1023u));
        }
        s_xs[lane] = xs;
        s_k[lane] = k;
    }
    __syncthreads();
    const int rec = T.rec, rec_words = (rec + 3) >> 2;
    uint8_t* cont = is_v ? a.v_cont : a.k_cont;
    for (int idx = threadIdx.x; idx < ns * rec_words * 4; idx += blockDim.x) {
        const int si = idx / (rec_words * 4), i = idx - si * rec_words * 4;
        const long long sid = first + si;
        const int sl = a.slot[(int)(sid / groups)], grp = (int)(sid % groups);
        const int k = (int)s_k[si], used = min(8 + k, rec);
        uint8_t v = 0;
        if (i < 4) v = (uint8_t)(s_hdr[si] >> (8 * i));
        else if (i < 8) v = (uint8_t)(s_xs[si] >> (8 * (i - 4)));
        else if (i < used) v = s_bytesT[(k - 1 - (i - 8)) * kWB + si];   // emitted last = read first
        uint8_t* blk = cont + ((size_t)(sl / DQ_PAGE_TOKENS) * groups + grp) * ((size_t)rec_words * 64) +
                       (size_t)(sl % DQ_PAGE_TOKENS) * 4;
        blk[(size_t)(i >> 2) * 64 + (i & 3)] = v;
    }
    if (threadIdx.x < ns) add_status(a.status, s_flags[threadIdx.x], (int)s_k[threadIdx.x]);
}

}  // namespace

cudaError_t dq_launch_means(const DqDevTable& tk, const void* k_bf16, int T, int Hkv,
                            const int32_t* seq_id, const int32_t* pos, int8_t* mean_q,
                            float* mean_scale, int max_windows, int mode, const float* rope_cos,
                            const float* rope_sin, int rope_style, cudaStream_t st) {
    if (T == 0 || Hkv == 0) return cudaSuccess;
    if (mode != DQ_MEAN_COMPUTE) return cudaSuccess;  // carry-forward is done by the encoder warps
    const unsigned blocks = (unsigned)((T + kMeansTokens - 1) / kMeansTokens);
    dq_means_compute_kernel<<<blocks, 256, 0, st>>>((const uint16_t*)k_bf16, T, Hkv, tk.rotate, seq_id, pos,
                                                    mean_q, mean_scale, max_windows, rope_cos, rope_sin, rope_style);
    return cudaGetLastError();
}

// Smallest number of streams for which a call goes to the batch kernels (32 streams per CTA); the
// option DQ_OPT_ENCODE_BATCH_MIN replaces the default (0 sends every call there).
static long long batch_min_streams(long long dflt) { return dq_opt_encode_batch_min(dflt); }

cudaError_t dq_launch_encode(const DqDevTable& tk, const DqDevTable& tv, const DqPairEnc& pk, const DqPairEnc& pv,
                             const DqEncodeArgs& a, cudaStream_t st) {
    const long long warps = (long long)a.T * a.Hkv;
    if (warps == 0 || (!a.do_k && !a.do_v)) return cudaSuccess;
    if (tk.hs > 1) {   // token-wide streams: CTAs of hs warps; few streams: one per CTA, many: 32 per CTA
        const long long streams = warps / tk.hs;
        const dim3 kinds_y(1, (a.do_k && a.do_v) ? 2 : 1);
        const bool wpair = tk.pair != 0;   // the caller has checked that both tables agree
        if (streams < batch_min_streams(3LL * 148 * kWB))
            return dq_launch_pdl(wpair ? dq_encode_wide_kernel<true> : dq_encode_wide_kernel<false>, dim3((unsigned)streams, kinds_y.y),
                                 dim3(tk.hs * 32), 0, st, tk, tv, pk, pv, a);
        const int smem = wide_batch_smem(tk.hs, tk.rec > tv.rec ? tk.rec : tv.rec);
        auto batch_kernel = wpair ? dq_encode_wide_batch_kernel<true> : dq_encode_wide_batch_kernel<false>;
        const cudaError_t e = cudaFuncSetAttribute(batch_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return e;
        return dq_launch_pdl(batch_kernel, dim3((unsigned)((streams + kWB - 1) / kWB), kinds_y.y),
                             dim3(tk.hs * 32), (size_t)smem, st, tk, tv, pk, pv, a);
    }
    const unsigned blocks = (unsigned)((warps + kEncWarps - 1) / kEncWarps);
    const bool pair = tk.pair != 0;   // the caller has checked that both tables agree
    const dim3 kinds(1, (a.do_k && a.do_v) ? 2 : 1);
    if (!a.step_flags && warps >= batch_min_streams(4LL * 148 * kB32 * 4))   // enough streams to fill the GPU several times
        return dq_launch_pdl(pair ? dq_encode_batch32_kernel<kB32PairMinBlocks, true> : dq_encode_batch32_kernel<DQ_B32_MINB, false>,
                             dim3((unsigned)((warps + kB32 - 1) / kB32), kinds.y), dim3(kB32Warps * 32), 0, st, tk, tv, pk, pv, a);
    if (a.step_flags) {   // decode step: big CTAs, so that few SMs are kept from the attention kernel
        constexpr int kStepWarps = DQ_STEP_ENC_WARPS;
        return dq_launch_pdl(pair ? dq_encode_kernel<1, kStepWarps, true> : dq_encode_kernel<1, kStepWarps, false>,
                             dim3((unsigned)((warps + kStepWarps - 1) / kStepWarps), kinds.y), dim3(kStepWarps * 32), 0, st, tk, tv, pk, pv, a);
    }
    return dq_launch_pdl(pair ? dq_encode_kernel<2, kEncWarps, true> : dq_encode_kernel<2, kEncWarps, false>, dim3(blocks, kinds.y),
                         dim3(kEncWarps * 32), 0, st, tk, tv, pk, pv, a);
}
