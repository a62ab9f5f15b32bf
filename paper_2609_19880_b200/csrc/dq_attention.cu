// Fused decode-step attention over rANS-coded KV containers (Sec. 4.5 "Decoding";
// Algorithm 2; Appendix A Eq. fold-key / fold-value) for sm_100a.
//
// Launch sequence per call (one stream):
//   dq_attn_prepare_kernel   rotate q (q' = H q / sqrt(128)), per-sequence block prefix
//                            sums, reset of the work counter
//   dq_attention_kernel      persistent, one CTA per SM; work items (sequence, KV head,
//                            block of NW*32 tokens) are dealt round-robin to the CTAs.  Each warp owns 32 tokens of the item: lane l runs the
//                            rANS state machine of token l out of shared memory, levels go to
//                            a small fp16 tile and from there into mma.sync contractions
//                            against q' (keys) and the softmax weights (values).  s, o and
//                            the window mean are applied after the contraction.  The loop is
//                            software-pipelined across items: while a warp decodes the K
//                            streams of item n it also decodes the V streams of item n-1
//                            (whose softmax weights are known), two independent dependency
//                            chains per lane; records of item n+1 arrive by cp.async.
//   dq_attn_combine_kernel   log-sum-exp merge of the per-item partials, inverse rotation
//                            of the output when V was rotated, bf16 / f32 store.
//
// The integer ALU pipe (half rate) is what binds the decode, so the per-symbol step is
// written to spread work over the pipes: table address and field extraction by dp4a (FMA
// pipe), renormalisation byte merged by one byte-permute, selector bumped by a mad.
// q' and the softmax weights enter the tensor cores as fp16 hi + lo pairs, so the
// contractions carry ~22 mantissa bits; levels 0..15 are exact in fp16.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "dq_attention_common.cuh"

using namespace dqdev;
using namespace dqattn;

namespace {

constexpr int kTileStride = 48;        // bytes per token row of a [32 tok][16 ch] fp16 tile; the
                                       // 16 pad bytes of the K tile rows hold (sK, oK, sV, oV)
constexpr int kTileBytes = kChunk * kTileStride;
constexpr int kKTail = 32;             // bytes after a warp's K records: q'.mean of its window, per head

struct Item {
    int b, h, blk, len, bg, valid;
    int late;   // decode-step mode: the block holds the sequence's newest token, whose record the step's encoder writes
    int pad1;
};

struct Layout {
    int stage_k, stage_v;               // bytes of one warp's K (+ tail) / V record buffer
    int off_lutk, off_lutv, off_prefix, off_q16, off_qsum, off_red, off_pages, off_items, off_kst, off_vst, off_tiles,
        off_obuf, total;
    int warp_tile_bytes, warp_obuf_bytes;
};

__host__ __device__ inline int align16(int x) { return (x + 15) & ~15; }

__host__ __device__ inline Layout make_layout(int nw, int rec_k, int rec_v, int B, int G) {
    Layout L;
    L.stage_k = align16(kChunk * rec_k) + kKTail;
    L.stage_v = align16(kChunk * rec_v);
    L.warp_tile_bytes = 2 * kTileBytes;             // K tile (+ per-token metadata), V tile
    L.warp_obuf_bytes = G * kORow * 4;              // this warp's O[g][channel], l, off
    // compile-time offsets first (the decode loop's addresses then cost no registers), sizes that
    // depend on the launch after them
    int o = 0;
    L.off_lutk = o; o += 256 * 32 * 4;
    L.off_lutv = o; o += 256 * 32 * 4;
    L.off_q16 = o; o += 2 * kQ16Bytes;
    L.off_qsum = o; o += 2 * DQ_MAX_GROUP * 4;
    L.off_red = o; o += (kMaxWarps + 2) * DQ_MAX_GROUP * 4;
    L.off_pages = o; o += kMaxWarps * 3 * 2 * 4 + 16;   // per warp: page ids of 3 items in flight; prev row
    L.off_items = o; o += 4 * 32;                       // descriptors of the items n .. n + 3 of this CTA
    L.off_tiles = o; o += nw * L.warp_tile_bytes;
    L.off_obuf = o; o += nw * L.warp_obuf_bytes;
    L.off_kst = o; o += 2 * nw * L.stage_k;
    L.off_vst = o; o += 2 * nw * L.stage_v;
    L.off_prefix = o; o += align16((3 * B + 2) * 4);   // block prefix sums, sequence lengths, non-empty counts
    L.total = o + 256;  // slack: a malformed record may be over-read by up to 136 + 8 bytes
    return L;
}

// ------------------------------------------------------------------ prepare

// Warp roles: [0, B*Hq): rotate q, emit the fp16 hi/lo operand rows and the row sum;
// then B*Hq warps per group of 8 windows: q' . mean of each (head, window) (Eq. fold-key, third
// term); block 0 additionally scans the blocks per sequence and resets the work counter.
constexpr int kPrepWindows = 8;
__global__ void __launch_bounds__(256)
dq_attn_prepare_kernel(AttnParams p) {
    pdl_launch_dependents();
    // Decode-step mode: this kernel was let go by the step's encoder after THAT kernel's wait, so everything
    // older is complete; it must not wait for the encoder (it runs beside it) and reads nothing the encoder writes.
    if (!p.fused) pdl_wait_prior_grid();   // q, the window means and seq_lens may come from the previous kernel
    const int lane = threadIdx.x & 31;
    const long long wid = (long long)blockIdx.x * 8 + (threadIdx.x >> 5);
    const int heads = p.B * p.Hq;
    const int wgroups = p.has_mean ? (p.windows + kPrepWindows - 1) / kPrepWindows : 0;
    if (wid < (long long)heads * (1 + wgroups)) {
        const int head = (int)(wid % heads), win = (int)(wid / heads) - 1;
        const uint2 raw = *reinterpret_cast<const uint2*>(p.q + qo_row(p, head / p.Hq, head % p.Hq) * kN + 4 * lane);
        float v[4] = {bf16_bits_to_float(raw.x & 0xffffu), bf16_bits_to_float(raw.x >> 16),
                      bf16_bits_to_float(raw.y & 0xffffu), bf16_bits_to_float(raw.y >> 16)};
        if (p.rotate_q) warp_fwht128(v, lane);
        const int b = head / p.Hq, hq = head % p.Hq, h = hq / p.G, g = hq % p.G;
        if (win < 0) {
            *reinterpret_cast<float4*>(p.qrot + (size_t)head * kN + 4 * lane) = make_float4(v[0], v[1], v[2], v[3]);
            uint16_t* rows = p.q16 + ((size_t)b * p.Hkv + h) * 16 * kN;
            __half hi[4], lo[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                hi[e] = __float2half_rn(v[e]);
                lo[e] = __float2half_rn(v[e] - __half2float(hi[e]));
            }
            uint2 w;
            w.x = (uint32_t)__half_as_ushort(hi[0]) | ((uint32_t)__half_as_ushort(hi[1]) << 16);
            w.y = (uint32_t)__half_as_ushort(hi[2]) | ((uint32_t)__half_as_ushort(hi[3]) << 16);
            *reinterpret_cast<uint2*>(rows + (size_t)g * kN + 4 * lane) = w;
            w.x = (uint32_t)__half_as_ushort(lo[0]) | ((uint32_t)__half_as_ushort(lo[1]) << 16);
            w.y = (uint32_t)__half_as_ushort(lo[2]) | ((uint32_t)__half_as_ushort(lo[3]) << 16);
            *reinterpret_cast<uint2*>(rows + (size_t)(8 + g) * kN + 4 * lane) = w;
            if (g == 0)  // unused operand rows of this KV head are zero
                for (int r = p.G; r < 8; ++r) {
                    *reinterpret_cast<uint2*>(rows + (size_t)r * kN + 4 * lane) = make_uint2(0u, 0u);
                    *reinterpret_cast<uint2*>(rows + (size_t)(8 + r) * kN + 4 * lane) = make_uint2(0u, 0u);
                }
            float s = (v[0] + v[1]) + (v[2] + v[3]);
#pragma unroll
            for (int d = 16; d >= 1; d >>= 1) s += __shfl_xor_sync(kFullMask, s, d);
            if (lane == 0) p.qsum[head] = s;
        } else {
            uint32_t q4[kPrepWindows];
            float msc[kPrepWindows], s[kPrepWindows];
            // Decode-step mode: when the newest token opens a window, the encoder is writing that window's
            // mean right now as a copy of the previous window's (zero for window 0): read the source instead.
            int w_open = -1;
            if (p.fused) {
                const int np = p.seq_lens[b] - 1;
                if (np >= 0 && np % DQ_WINDOW_TOKENS == 0) w_open = np / DQ_WINDOW_TOKENS;
            }
#pragma unroll
            for (int u = 0; u < kPrepWindows; ++u) {   // all loads first
                const int w = min(win * kPrepWindows + u, p.windows - 1);
                const int ws = (w == w_open) ? w - 1 : w;
                const size_t mi = ((size_t)b * p.max_windows + max(ws, 0)) * p.Hkv + h;
                q4[u] = *reinterpret_cast<const uint32_t*>(p.mean_q + mi * kN + 4 * lane);
                msc[u] = ws < 0 ? 0.f : p.mean_scale[mi];
            }
#pragma unroll
            for (int u = 0; u < kPrepWindows; ++u) {
                s[u] = 0.f;
#pragma unroll
                for (int e = 0; e < 4; ++e) s[u] = fmaf(v[e], msc[u] * (float)(int)(int8_t)((q4[u] >> (8 * e)) & 0xffu), s[u]);
            }
#pragma unroll
            for (int d = 16; d >= 1; d >>= 1)
#pragma unroll
                for (int u = 0; u < kPrepWindows; ++u) s[u] += __shfl_xor_sync(kFullMask, s[u], d);
#pragma unroll
            for (int u = 0; u < kPrepWindows; ++u)
                if (lane == u && win * kPrepWindows + u < p.windows) p.qmu[(size_t)head * p.windows + win * kPrepWindows + u] = s[u];
        }
    }
    if (blockIdx.x == 0 && threadIdx.x < 32) {  // exclusive scans: blocks per sequence, non-empty sequences
        int carry = 0, ne_carry = 0;
        for (int base = 0; base < p.B; base += 32) {
            const int b = base + lane;
            int nb = 0;
            if (b < p.B) nb = (min(max(p.seq_lens[b], 0), p.max_pages * DQ_PAGE_TOKENS) + p.item_tokens - 1) / p.item_tokens;
            int incl = nb, ne = nb > 0 ? 1 : 0;
            const int ne_self = ne;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const int o = __shfl_up_sync(kFullMask, incl, d), oe = __shfl_up_sync(kFullMask, ne, d);
                if (lane >= d) { incl += o; ne += oe; }
            }
            if (b < p.B) { p.prefix[b] = carry + incl - nb; p.ne_before[b] = ne_carry + ne - ne_self; }
            carry += __shfl_sync(kFullMask, incl, 31);
            ne_carry += __shfl_sync(kFullMask, ne, 31);
        }
        if (lane == 0) { p.prefix[p.B] = carry; p.ne_before[p.B] = ne_carry; if (!p.fused) *p.counter = 0; }
    }
    if (p.fused) {
        // Hand-over: when the last CTA is done, it publishes the first dynamic item index (the first three
        // items of every attention CTA are dealt statically) and then the ready flag, and one of its threads
        // stays to wait for the encoder, so that this kernel's end implies the encoder's.  Every other CTA
        // leaves at once: the attention CTAs need whole SMs.
        __threadfence();
        __syncthreads();
        if (threadIdx.x == 0 && atomicAdd(&p.flags[2], 1) == (int)gridDim.x - 1) {
            p.flags[0] = 3 * p.attn_grid;
            __threadfence();
            atomicExch(&p.flags[1], 1);
            pdl_wait_prior_grid();
        }
    }
}

// --------------------------------------------------------------------- main

// Decode 16 symbols of one stream (Algorithm 2) and pack their levels as 8 fp16x2 words.
//   x    rANS state;  ptr  shared-memory byte address of the next renormalisation byte
//   lut  shared address of this lane's column of the 32-way replicated table: entry z at
//        lut + 128 z, entry = f << 24 | fp16(level) << 8 | (z - c)
//   one  the value 1 in a register (keeps the selector bump a multiply-add)
// Per symbol: z = x mod 256 addresses the table (dp4a: 128 * byte0(x) + lut); x = f * (x >> 8)
// + (z - c) (f by dp4a, product by mad, addend by dp4a); if x < L one byte is appended with a
// byte-permute from a 4-byte window that is reloaded every 4 symbols (a symbol takes at most
// one byte because the state stays >= 2^15).
// LBITS: log2 of the lower bound L of the state interval, 23 (32-bit final state) or 15 (24-bit).
template <int LBITS>
__device__ __forceinline__ void decode16(uint32_t& x, uint32_t& ptr, uint32_t lut, uint32_t one,
                                         uint32_t (&packed)[8]) {
#pragma unroll
    for (int q4 = 0; q4 < 4; ++q4) {
        const uint32_t base = ptr & ~3u;
        const uint32_t win = __funnelshift_r(lds32(base), lds32(base + 4), ptr << 3);
        uint32_t sel = 0x2104u;
        uint32_t e[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            e[i] = lds32(dp4a_u32(x, 0x80u, lut));
            const uint32_t f = dp4a_u32(e[i], 0x01000000u, 0u);
            const uint32_t t = f * (x >> 8);
            x = dp4a_u32(e[i], 1u, t);
            asm("{.reg .pred p; setp.lt.u32 p, %0, %4; @p prmt.b32 %0, %0, %2, %1; "
                "@p mad.lo.u32 %1, %3, %3, %1;}"
                : "+r"(x), "+r"(sel) : "r"(win), "r"(one), "n"(1u << LBITS));
        }
        ptr += sel - 0x2104u;
        packed[2 * q4] = __byte_perm(e[0], e[1], 0x6521u);
        packed[2 * q4 + 1] = __byte_perm(e[2], e[3], 0x6521u);
    }
}

// Paired-symbol variant: one step decodes the levels of two consecutive channels, 8 steps the 16.  A table
// entry is code(b) << 24 | f << 16 | code(a) << 8 | (z - c) with code(m) the high byte of the fp16
// pattern of level m (levels 0..8 have a zero low byte), so a step's fp16x2 word (level a, level b) is the
// entry with its f and (z - c) bytes cleared.
template <int LBITS>
__device__ __forceinline__ void decode16_pairs(uint32_t& x, uint32_t& ptr, uint32_t lut, uint32_t one,
                                               uint32_t (&packed)[8]) {
#pragma unroll
    for (int q4 = 0; q4 < 2; ++q4) {
        const uint32_t base = ptr & ~3u;
        const uint32_t win = __funnelshift_r(lds32(base), lds32(base + 4), ptr << 3);
        uint32_t sel = 0x2104u;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint32_t e = lds32(dp4a_u32(x, 0x80u, lut));
            const uint32_t f = dp4a_u32(e, 0x00010000u, 0u);
            const uint32_t t = f * (x >> 8);
            x = dp4a_u32(e, 1u, t);
            asm("{.reg .pred p; setp.lt.u32 p, %0, %4; @p prmt.b32 %0, %0, %2, %1; "
                "@p mad.lo.u32 %1, %3, %3, %1;}"
                : "+r"(x), "+r"(sel) : "r"(win), "r"(one), "n"(1u << LBITS));
            packed[4 * q4 + i] = e & 0xff00ff00u;
        }
        ptr += sel - 0x2104u;
    }
}

// One pass over the 128 channels, 16 at a time.  With DO_K the K streams of the current item
// are decoded and S[g][t] = sum_j q'_gj level_tj accumulated (Eq. fold-key, inner sum).  With
// DO_V the V streams of the previous item are decoded and each finished 16-channel tile of
// O[j][g] = sum_t (a_t s_t) level_tj (Eq. fold-value, first sum) goes to this warp's output
// slot in shared memory.  Both decodes are interleaved in one instruction stream.
template <bool DO_K, bool DO_V, int LBITS, bool PAIRS>
__device__ __forceinline__ void fused_pass(uint32_t xk, uint32_t ptrk, uint32_t xv, uint32_t ptrv, uint32_t lutk,
                                           uint32_t lutv, uint32_t one, uint32_t ktile, uint32_t vtile, uint32_t q16,
                                           uint32_t obuf, int lane, int G, float (&sacc)[4][4],
                                           const uint32_t (&pb_hi)[2][2], const uint32_t (&pb_lo)[2][2]) {
    const uint32_t a_addr = q16 + ((lane & 7) + ((lane >> 3) & 1) * 8) * kQ16Stride + (lane >> 4) * 16;
    const uint32_t bk_addr = ktile + ((lane & 7) + (lane >> 4) * 8) * kTileStride + ((lane >> 3) & 1) * 16;
    const uint32_t av_addr = vtile + ((lane & 7) + (lane >> 4) * 8) * kTileStride + ((lane >> 3) & 1) * 16;
    // output slot: thread holds channels (lane/4, lane/4 + 8) of heads (2 qd, 2 qd + 1)
    const uint32_t o_addr = obuf + ((2 * (lane & 3)) * kORow + (lane >> 2)) * 4;
#ifndef DQ_EXP_CG
#define DQ_EXP_CG 8   // channel groups per pass (only ever changed to count the pass's instructions)
#endif
#pragma unroll 1
    for (int cg = 0; cg < DQ_EXP_CG; ++cg) {
        uint32_t pk[8], pv[8];
        if (DO_K) { if (PAIRS) decode16_pairs<LBITS>(xk, ptrk, lutk, one, pk); else decode16<LBITS>(xk, ptrk, lutk, one, pk); }
        if (DO_V) { if (PAIRS) decode16_pairs<LBITS>(xv, ptrv, lutv, one, pv); else decode16<LBITS>(xv, ptrv, lutv, one, pv); }
        if (DO_K) { sts128(ktile + lane * kTileStride, pk); sts128(ktile + lane * kTileStride + 16, pk + 4); }
        if (DO_V) { sts128(vtile + lane * kTileStride, pv); sts128(vtile + lane * kTileStride + 16, pv + 4); }
        __syncwarp();
        if (DO_K) {
            uint32_t a[4], b0[4], b1[4];
            ldmatrix_x4(a, a_addr + cg * 32);
            ldmatrix_x4(b0, bk_addr);
            ldmatrix_x4(b1, bk_addr + 16 * kTileStride);
            mma_f16_16816(sacc[0], a, b0[0], b0[1]);
            mma_f16_16816(sacc[1], a, b0[2], b0[3]);
            mma_f16_16816(sacc[2], a, b1[0], b1[1]);
            mma_f16_16816(sacc[3], a, b1[2], b1[3]);
        }
        if (DO_V) {
            uint32_t a0[4], a1[4];
            float o[4] = {0.f, 0.f, 0.f, 0.f};
            ldmatrix_x4_trans(a0, av_addr);                      // tokens 0..15, 16 channels
            ldmatrix_x4_trans(a1, av_addr + 16 * kTileStride);   // tokens 16..31
            mma_f16_16816(o, a0, pb_hi[0][0], pb_hi[0][1]);
            mma_f16_16816(o, a1, pb_hi[1][0], pb_hi[1][1]);
            mma_f16_16816(o, a0, pb_lo[0][0], pb_lo[0][1]);
            mma_f16_16816(o, a1, pb_lo[1][0], pb_lo[1][1]);
            const uint32_t oa = o_addr + cg * 64;
            if (2 * (lane & 3) < G) { sts32f(oa, o[0]); sts32f(oa + 32, o[2]); }
            if (2 * (lane & 3) + 1 < G) { sts32f(oa + kORow * 4, o[1]); sts32f(oa + kORow * 4 + 32, o[3]); }
        }
        __syncwarp();
    }
}

// FUSED (decode-step mode): the kernel starts while the step's encoder still runs.  It takes the
// prepare kernel's outputs on a ready flag instead of waiting for that kernel, pulls its work items
// from a global counter (SMs still busy with the encoder join late and simply take fewer), leaves the
// blocks that hold a sequence's newest token to the end of the item order, and waits for the preceding
// kernels -- whose completion implies the encoder's -- only before the first of those blocks.
#ifndef DQ_STEP_POLL_LIMIT
#define DQ_STEP_POLL_LIMIT (1 << 16)   // polls of the ready flag (64 ns apart) before a CTA falls back to the grid wait
#endif
// The option DQ_OPT_STEP_POLL_LIMIT replaces the default; 0 makes every CTA take the fallback at once,
// which is how the tests run that path.
static int step_poll_limit() { return dq_opt_step_poll_limit(DQ_STEP_POLL_LIMIT); }
// PAIRS: the tables' rANS symbols are pairs of levels (64 steps per stream instead of 128).
template <bool FUSED, int LBITS, bool PAIRS>
__global__ void __launch_bounds__(kMaxWarps * 32, 1)
dq_attention_kernel(const __grid_constant__ DqDevTable TK, const __grid_constant__ DqDevTable TV,
                    const AttnParams p) {
    extern __shared__ __align__(128) uint8_t smem[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nthreads = blockDim.x, nw = nthreads >> 5;
    const int G = p.G;
    const Layout L = make_layout(nw, TK.rec, TV.rec, p.B, G);
    const uint32_t sbase = smem_addr(smem);

    uint32_t* lutk = reinterpret_cast<uint32_t*>(smem + L.off_lutk);
    uint32_t* lutv = reinterpret_cast<uint32_t*>(smem + L.off_lutv);
    int* prefix = reinterpret_cast<int*>(smem + L.off_prefix);      // [B + 1] blocks before sequence b
    int* s_len = prefix + (p.B + 1);                                // [B] clamped sequence lengths
    float* qsum = reinterpret_cast<float*>(smem + L.off_qsum);      // [2][8]
    float* red_m = reinterpret_cast<float*>(smem + L.off_red);      // [warp][head] chunk maxima
    float* red_M = red_m + kMaxWarps * DQ_MAX_GROUP;                // [2][head] item maxima
    float* obuf_all = reinterpret_cast<float*>(smem + L.off_obuf);  // [warp][head][kORow]

    pdl_launch_dependents();
    for (int i = tid; i < 256 * 32; i += nthreads) {   // tables come from the kernel parameters
        lutk[i] = TK.lut[i >> 5];
        lutv[i] = TV.lut[i >> 5];
    }
    int* ne_before = s_len + p.B;                                   // [B + 1] (FUSED) non-empty sequences before b
    bool waited = !FUSED;   // the preceding kernels are known to be complete
    if (FUSED) {
        // acquire-poll the ready flag (bounded); a CTA that gives up waits for the preceding kernels instead
        int* s_ok = reinterpret_cast<int*>(smem + L.off_items);
        if (tid == 0) {
            int ok = 0;
            for (int it = 0; it < p.poll_limit && !ok; ++it) {
                asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(ok) : "l"(p.flags + 1) : "memory");
                if (!ok) __nanosleep(64);
            }
            if (!ok) atomicAdd(p.flags + 3, 1);
            *s_ok = ok;
        }
        __syncthreads();
        if (!*s_ok) { pdl_wait_prior_grid(); waited = true; }
        __syncthreads();
    } else {
        pdl_wait_prior_grid();   // everything below reads what the prepare kernel wrote
    }
    for (int i = tid; i <= p.B; i += nthreads) {
        prefix[i] = p.prefix[i];
        if (i < p.B) s_len[i] = min(p.seq_lens[i], p.max_pages * DQ_PAGE_TOKENS);
        if (FUSED) ne_before[i] = p.ne_before[i];
    }
    __syncthreads();
    const int total_items = prefix[p.B] * p.Hkv;

    const uint32_t my_lutk = sbase + L.off_lutk + lane * 4, my_lutv = sbase + L.off_lutv + lane * 4;
    const uint32_t ktile = sbase + L.off_tiles + warp * L.warp_tile_bytes, vtile = ktile + kTileBytes;
    const uint32_t my_obuf = sbase + L.off_obuf + warp * L.warp_obuf_bytes;
    const uint32_t one = (sbase >> 31) | 1u;
    const int g_row = lane >> 2, qd = lane & 3;

    // Items are dealt round-robin to the CTAs.  Thread 0 derives the descriptor of item n + 3 while the
    // CTA works on item n and leaves it in a ring of four in shared memory; everybody else reads the
    // descriptors it needs (n, n + 1, n + 2) after the next CTA barrier, so neither a global atomic nor
    // the search sits on the critical path.  (Item indices of one CTA grow with n, so the sequence is
    // found by walking forward from `hint`, the sequence of an earlier item.)
    auto item_of = [&](int n, int hint) {
        Item it;
        it.valid = 0; it.b = hint; it.h = it.blk = it.len = it.bg = 0; it.late = it.pad1 = 0;
        const unsigned idx = blockIdx.x + (unsigned)n * gridDim.x;   // < 2^31: total_items is an int
        if (idx < (unsigned)total_items) {
            it.valid = 1;
            // idx / Hkv by a high multiply: exact for idx < 2^32 / Hkv (hkv_magic = ceil(2^32 / Hkv); 0: Hkv = 1)
            it.bg = p.hkv_magic ? (int)__umulhi(idx, p.hkv_magic) : (int)idx;
            it.h = (int)(idx - (unsigned)it.bg * (unsigned)p.Hkv);
            int b = hint;
            while (prefix[b + 1] <= it.bg) ++b;   // prefix[B] > bg because idx < total_items
            it.b = b;
            it.blk = it.bg - prefix[b];
            it.len = s_len[b];
        }
        return it;
    };
    // Decode-step mode: item order = every block that is not the last of its sequence (sequence-major),
    // then the last blocks; the first three items of a CTA are static, the rest come from the counter.
    int hint = 0;        // thread 0: sequence of the newest descriptor, the search start for the next one
    int hint_late = 0;   // thread 0: search start among the last blocks
    auto item_of_fused = [&](int n) {
        Item it;
        it.valid = 0; it.b = 0; it.h = it.blk = it.len = it.bg = 0; it.late = it.pad1 = 0;
        const int n_early = (prefix[p.B] - ne_before[p.B]) * p.Hkv, n_late = ne_before[p.B] * p.Hkv;
        unsigned r;
        if (n < 3) r = blockIdx.x + (unsigned)n * gridDim.x;
        else r = (unsigned)atomicAdd(p.flags + 0, 1);
        if (r >= (unsigned)(n_early + n_late)) return it;
        it.valid = 1;
        if (r < (unsigned)n_early) {
            const int bgA = p.hkv_magic ? (int)__umulhi(r, p.hkv_magic) : (int)r;   // r / Hkv
            it.h = (int)(r - (unsigned)bgA * (unsigned)p.Hkv);
            int b = hint;   // non-last blocks before sequence b: prefix[b] - ne_before[b]
            while (prefix[b + 1] - ne_before[b + 1] <= bgA) ++b;
            hint = b;
            it.b = b;
            it.blk = bgA - (prefix[b] - ne_before[b]);
        } else {
            const unsigned rl = r - (unsigned)n_early;
            const int j = p.hkv_magic ? (int)__umulhi(rl, p.hkv_magic) : (int)rl;   // j-th non-empty sequence
            it.h = (int)(rl - (unsigned)j * (unsigned)p.Hkv);
            int b = hint_late;
            while (ne_before[b + 1] <= j) ++b;
            hint_late = b;
            it.b = b;
            it.blk = prefix[b + 1] - prefix[b] - 1;
            it.late = 1;
        }
        it.bg = prefix[it.b] + it.blk;
        it.len = s_len[it.b];
        return it;
    };
    // The physical page ids of this warp's 32 tokens are fetched two items ahead by cp.async into
    // a small ring in shared memory (slot n % 3), so neither their latency nor registers are spent.
    int* my_pages = reinterpret_cast<int*>(smem + L.off_pages) + warp * 6;
    long long* s_prev_row = reinterpret_cast<long long*>(smem + L.off_pages + kMaxWarps * 24);
    auto fetch_pages = [&](int n, const Item& it) {
        const int tok0 = (it.blk * nw + warp) * kChunk;
        if (it.valid && tok0 < it.len && lane < 2 && tok0 + 16 * lane < it.len)
            cp_async4(smem_addr(my_pages + (n % 3) * 2 + lane),
                      p.page_table + (size_t)it.b * p.max_pages + (tok0 >> 4) + lane);
    };
    // cp.async of the K records, q'.mean values and q' operand of item n_k, V records of item n_v.
    // A warp's 32 tokens are two pages whose (page, head) blocks land back to back in its buffer, so
    // piece i of the 2 * rec 16-byte pieces goes to buffer offset 16 i and comes from page i / rec.
    auto issue_loads = [&](int nk, const Item& ik, int nv, const Item& iv) {
        if (ik.valid) {
            const int tok0 = (ik.blk * nw + warp) * kChunk;
            if (tok0 < ik.len) {
                const uint32_t kst = sbase + L.off_kst + ((nk & 1) * nw + warp) * L.stage_k;
                const int rec = TK.rec, np = (tok0 + 16 < ik.len) ? 2 * rec : rec;
                const uint32_t blk = 16u * (uint32_t)rec;
                const uint8_t* s0 = p.k_cont + ((size_t)my_pages[(nk % 3) * 2] * p.Hkv + ik.h) * blk;
                const uint8_t* s1 = p.k_cont + ((size_t)my_pages[(nk % 3) * 2 + 1] * p.Hkv + ik.h) * blk - blk;
                for (int i = lane; i < np; i += 32) cp_async16(kst + i * 16, (i < rec ? s0 : s1) + i * 16);
                if (p.has_mean && lane < G)
                    cp_async4(kst + L.stage_k - kKTail + lane * 4,
                              p.qmu + ((size_t)ik.b * p.Hq + (size_t)ik.h * G + lane) * p.windows + tok0 / DQ_WINDOW_TOKENS);
            }
            if (tid < 16 * 16) {   // q' operand: 16 rows x 16 pieces of 16 bytes
                const uint16_t* qsrc = p.q16 + ((size_t)ik.b * p.Hkv + ik.h) * 16 * kN;
                for (int i = tid; i < 16 * 16; i += nthreads)
                    cp_async16(sbase + L.off_q16 + (nk & 1) * kQ16Bytes + (i >> 4) * kQ16Stride + (i & 15) * 16, qsrc + i * 8);
                if (tid < G)
                    cp_async4(sbase + L.off_qsum + ((nk & 1) * DQ_MAX_GROUP + tid) * 4,
                              p.qsum + (size_t)ik.b * p.Hq + (size_t)ik.h * G + tid);
            }
        }
        if (iv.valid) {
            const int tok0 = (iv.blk * nw + warp) * kChunk;
            if (tok0 < iv.len) {
                const uint32_t vst = sbase + L.off_vst + ((nv & 1) * nw + warp) * L.stage_v;
                const int rec = TV.rec, np = (tok0 + 16 < iv.len) ? 2 * rec : rec;
                const uint32_t blk = 16u * (uint32_t)rec;
                const uint8_t* s0 = p.v_cont + ((size_t)my_pages[(nv % 3) * 2] * p.Hkv + iv.h) * blk;
                const uint8_t* s1 = p.v_cont + ((size_t)my_pages[(nv % 3) * 2 + 1] * p.Hkv + iv.h) * blk - blk;
                for (int i = lane; i < np; i += 32) cp_async16(vst + i * 16, (i < rec ? s0 : s1) + i * 16);
            }
        }
    };

    Item* s_items = reinterpret_cast<Item*>(smem + L.off_items);
    if (tid == 0) {
        for (int n = 0; n < 3; ++n) {
            if (FUSED) { s_items[n] = item_of_fused(n); continue; }
            const Item it = item_of(n, hint);
            s_items[n] = it;
            hint = it.b;
        }
    }
    __syncthreads();
    // prologue: page ids of items 0 and 1, then the K records of item 0
    {
        const Item i0 = s_items[0];
        if (FUSED && !waited && i0.valid && i0.late) { pdl_wait_prior_grid(); waited = true; }
        fetch_pages(0, i0);
        fetch_pages(1, s_items[1]);
        cp_async_commit();
        cp_async_wait<0>();
        __syncwarp();
        Item none = i0; none.valid = 0;
        issue_loads(0, i0, 0, none);
        cp_async_commit();
    }

    // state carried from the item whose V streams are still to be decoded
    bool have_prev = false;
    uint32_t pb_hi[2][2] = {{0u, 0u}, {0u, 0u}}, pb_lo[2][2] = {{0u, 0u}, {0u, 0u}};

    for (int n = 0;; ++n) {
        Item cur = s_items[n & 3];
        if (!cur.valid && !have_prev) break;
        {   // records of item n + 1 (its page ids arrived last iteration), page ids of item n + 2
            if (FUSED && !waited && s_items[(n + 1) & 3].valid && s_items[(n + 1) & 3].late) {
                pdl_wait_prior_grid();   // the newest tokens' records are complete from here on
                waited = true;
            }
            issue_loads(n + 1, s_items[(n + 1) & 3], n, cur);
            fetch_pages(n + 2, s_items[(n + 2) & 3]);
            cp_async_commit();
        }
        cp_async_wait<1>();
        __syncthreads();   // q' operand of `cur` visible; last iteration's merge reads are done
        if (tid == 0) {    // slot of item n - 1, which nobody reads any more
            if (FUSED) {
                s_items[(n + 3) & 3] = item_of_fused(n + 3);
            } else {
                const Item it = item_of(n + 3, hint);
                s_items[(n + 3) & 3] = it;
                hint = it.b;
            }
        }

        // ------------------------------------------ K streams of `cur`, V streams of `prev`
        int tok0 = (cur.blk * nw + warp) * kChunk;
        uint32_t kst = sbase + L.off_kst + ((n & 1) * nw + warp) * L.stage_k;
        const uint32_t vst_prev = sbase + L.off_vst + (((n + 1) & 1) * nw + warp) * L.stage_v;
        uint32_t rk = kst + lane * TK.rec;
        const uint32_t rvp = vst_prev + lane * TV.rec;
        const uint32_t q16 = sbase + L.off_q16 + (n & 1) * kQ16Bytes;
        float sacc[4][4];
#pragma unroll
        for (int i = 0; i < 4; ++i) { sacc[i][0] = sacc[i][1] = sacc[i][2] = sacc[i][3] = 0.f; }
        {
            // final state: 4 bytes (LBITS 23) or 3 bytes (LBITS 15) after the two fp16 grid parameters
            constexpr uint32_t kStateMask = LBITS == 23 ? 0xffffffffu : 0x00ffffffu;
            constexpr uint32_t kPay = LBITS == 23 ? 8u : 7u;
            const uint32_t xk = lds32_unaligned(rk + 4) & kStateMask, xv = lds32_unaligned(rvp + 4) & kStateMask;
            if (cur.valid && have_prev)
                fused_pass<true, true, LBITS, PAIRS>(xk, rk + kPay, xv, rvp + kPay, my_lutk, my_lutv, one, ktile, vtile, q16, my_obuf,
                                              lane, G, sacc, pb_hi, pb_lo);
            else if (cur.valid)
                fused_pass<true, false, LBITS, PAIRS>(xk, rk + kPay, xv, rvp + kPay, my_lutk, my_lutv, one, ktile, vtile, q16, my_obuf,
                                               lane, G, sacc, pb_hi, pb_lo);
            else
                fused_pass<false, true, LBITS, PAIRS>(xk, rk + kPay, xv, rvp + kPay, my_lutk, my_lutv, one, ktile, vtile, q16, my_obuf,
                                               lane, G, sacc, pb_hi, pb_lo);
        }

        // ------------------------------------------ logits of `cur` and this warp's maximum (base 2)
        cur = s_items[n & 3];   // read again rather than kept in registers across the pass
        tok0 = (cur.blk * nw + warp) * kChunk;
        kst = sbase + L.off_kst + ((n & 1) * nw + warp) * L.stage_k;
        rk = kst + lane * TK.rec;
        float lg[4][2], sv_t[4][2], ov_t[4][2];
        if (cur.valid) {
            cp_async_wait<0>();   // the V records of `cur` (header needed now) have landed
            __syncwarp();
            const uint32_t rv = sbase + L.off_vst + ((n & 1) * nw + warp) * L.stage_v + lane * TV.rec;
            {
                const uint32_t hk = lds32_unaligned(rk), hv = lds32_unaligned(rv);
                const float sK = __half2float(__ushort_as_half((unsigned short)(hk & 0xffffu)));
                const float oK = __half2float(__ushort_as_half((unsigned short)(hk >> 16)));
                const float sV = __half2float(__ushort_as_half((unsigned short)(hv & 0xffffu)));
                const float oV = __half2float(__ushort_as_half((unsigned short)(hv >> 16)));
                // the key scale carries the logit scale (sm_scale * log2 e): logits come out in base-2 units
                asm volatile("st.shared.v4.f32 [%0], {%1,%2,%3,%4};\n" ::"r"(ktile + lane * kTileStride + 32),
                             "f"(sK * p.scale_log2), "f"(oK), "f"(sV), "f"(oV) : "memory");
            }
            // tokens this thread's row may see: a query token that is not the last one stops earlier; tokens
            // of a BF16 residual window come after the compressed ones and absorb the offset first
            int row_len = cur.len;
            if (p.q_total > 1) row_len -= max(0, row_offset(p, g_row) - (p.resid_lens ? max(p.resid_lens[cur.b], 0) : 0));
            float qmu = 0.f, qs = 0.f;   // q' . window mean and sum of q' (both times the logit scale), for this thread's head row
            if (g_row < G) {
                qs = qsum[(n & 1) * DQ_MAX_GROUP + g_row] * p.scale_log2;
                if (p.has_mean && tok0 < cur.len) qmu = __uint_as_float(lds32(kst + L.stage_k - kKTail + g_row * 4)) * p.scale_log2;
            }
            __syncwarp();
            float mx = -INFINITY;
            const uint32_t meta = ktile + 2 * qd * kTileStride + 32;
            if (tok0 + kChunk <= row_len) {   // every token of the chunk is visible: no masks
#pragma unroll
                for (int i = 0; i < 4; ++i)
#pragma unroll
                    for (int u = 0; u < 2; ++u) {
                        float4 m4;
                        asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];\n"
                                     : "=f"(m4.x), "=f"(m4.y), "=f"(m4.z), "=f"(m4.w) : "r"(meta + (8 * i + u) * kTileStride));
                        lg[i][u] = fmaf(m4.x, sacc[i][u] + sacc[i][2 + u], fmaf(m4.y, qs, qmu));
                        sv_t[i][u] = m4.z;
                        ov_t[i][u] = m4.w;
                        mx = fmaxf(mx, lg[i][u]);
                    }
            } else {
                const int lim = row_len - tok0 - 2 * qd;   // token 8 i + 2 qd + u is visible iff 8 i + u < lim
#pragma unroll
                for (int i = 0; i < 4; ++i)
#pragma unroll
                    for (int u = 0; u < 2; ++u) {
                        float4 m4;
                        asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];\n"
                                     : "=f"(m4.x), "=f"(m4.y), "=f"(m4.z), "=f"(m4.w) : "r"(meta + (8 * i + u) * kTileStride));
                        const bool ok = 8 * i + u < lim;
                        lg[i][u] = ok ? fmaf(m4.x, sacc[i][u] + sacc[i][2 + u], fmaf(m4.y, qs, qmu)) : -INFINITY;
                        sv_t[i][u] = ok ? m4.z : 0.f;
                        ov_t[i][u] = ok ? m4.w : 0.f;
                        mx = fmaxf(mx, lg[i][u]);
                    }
            }
            mx = fmaxf(mx, __shfl_xor_sync(kFullMask, mx, 1));
            mx = fmaxf(mx, __shfl_xor_sync(kFullMask, mx, 2));
            if (qd == 0) red_m[warp * DQ_MAX_GROUP + g_row] = mx;
        }
        __syncthreads();   // output slots of `prev` complete; chunk maxima of `cur` published

        // ------------------------------------------ finish `prev`: sum its warps' slots, write the partial
        if (have_prev) {
            // G x 32 threads add the channel sums four at a time, 2 G more the (l, off) columns written when
            // `prev` was `cur` (by item parity); the item maximum goes along
            const int par = (n + 1) & 1;
            const int wstride = G * kORow;   // floats between the slots of neighbouring warps
            for (int e = tid; e < G * 34; e += nthreads) {
                if (e < G * 32) {
                    const int g = e >> 5, c4 = e & 31;
                    const float* src = obuf_all + g * kORow + 4 * c4;
                    float4 acc = *reinterpret_cast<const float4*>(src);
                    for (int w = 1; w < nw; ++w) {
                        const float4 v = *reinterpret_cast<const float4*>(src + w * wstride);
                        acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
                    }
                    *reinterpret_cast<float4*>(p.partial + ((size_t)s_prev_row[par] + g) * kPartial + 4 * c4) = acc;
                } else {
                    const int e2 = e - G * 32, g = e2 >> 1, which = e2 & 1;
                    const float* src = obuf_all + g * kORow + kN + 2 * par + which;
                    float acc = 0.f;
                    for (int w = 0; w < nw; ++w) acc += src[w * wstride];
                    float* dst = p.partial + ((size_t)s_prev_row[par] + g) * kPartial;
                    dst[kN + 1 + which] = acc;                   // l at 129, off at 130
                    if (which == 0) dst[kN] = red_M[par * DQ_MAX_GROUP + g];
                }
            }
        }

        // ------------------------------------------ softmax weights of `cur`, scaled by the item maximum
        have_prev = cur.valid;
        if (cur.valid) {
            float m_item = -INFINITY;   // the four threads of a head row share the warps' maxima
            for (int w = qd; w < nw; w += 4) m_item = fmaxf(m_item, red_m[w * DQ_MAX_GROUP + g_row]);
            m_item = fmaxf(m_item, __shfl_xor_sync(kFullMask, m_item, 1));
            m_item = fmaxf(m_item, __shfl_xor_sync(kFullMask, m_item, 2));
            if (warp == 0 && qd == 0) red_M[(n & 1) * DQ_MAX_GROUP + g_row] = m_item;
            const float m_use = (m_item == -INFINITY) ? 0.f : m_item;
            float lsum = 0.f, osum = 0.f;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                float ps[2];
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                    const float pr = ex2_approx(lg[i][u] - m_use);   // <= 1; exp2(-inf) = 0
                    lsum += pr;
                    osum = fmaf(pr, ov_t[i][u], osum);
                    ps[u] = pr * sv_t[i][u];
                }
                // fp16 hi + lo pair of each weight: hi = rn(ps), lo = rn(ps - hi)
                const __half2 h2 = __floats2half2_rn(ps[0], ps[1]);
                const float2 hf = __half22float2(h2);
                pb_hi[i >> 1][i & 1] = *reinterpret_cast<const uint32_t*>(&h2);
                pb_lo[i >> 1][i & 1] = pack_half2(ps[0] - hf.x, ps[1] - hf.y);
            }
            lsum += __shfl_xor_sync(kFullMask, lsum, 1);
            lsum += __shfl_xor_sync(kFullMask, lsum, 2);
            osum += __shfl_xor_sync(kFullMask, osum, 1);
            osum += __shfl_xor_sync(kFullMask, osum, 2);
            if (qd == 0 && g_row < G) {   // l and off ride along in this warp's output slot (columns by parity)
                sts32f(my_obuf + (g_row * kORow + kN + 2 * (n & 1)) * 4, lsum);
                sts32f(my_obuf + (g_row * kORow + kN + 2 * (n & 1) + 1) * 4, osum);
            }
        }
        if (tid == 0) s_prev_row[n & 1] = (long long)cur.bg * p.Hq + (long long)cur.h * G;   // read after two barriers
    }
    cp_async_wait<0>();
    // decode-step mode: no CTA leaves before the preceding kernels are complete, so that this kernel's end
    // implies theirs whatever the item mix was (returns at once by now)
    if (FUSED && !waited) pdl_wait_prior_grid();
}

// ------------------------------------------------------------------ combine

// One CTA of 8 warps per (sequence, query head): warp w merges partials w*4 .. w*4+3, w*4+32 ...
// with a running maximum, the warps are merged through shared memory, warp 0 normalises,
// applies the inverse rotation and stores.  With a BF16 residual window (Sec. 5.1: the most
// recent tokens stay uncompressed) the 8 warps also split those tokens: logits q.k and
// sum a_t v_t in the unrotated domain, merged with the un-rotated compressed part by the same
// log-sum-exp rule.
__global__ void __launch_bounds__(256)
dq_attn_combine_kernel(AttnParams p) {
    pdl_launch_dependents();
    pdl_wait_prior_grid();
    __shared__ float s_acc[8][kN];
    __shared__ float s_racc[8][kN];
    __shared__ float s_mlo[8][8];
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const int wid = blockIdx.x;
    const int b = wid / p.Hq, hq = wid % p.Hq;
    const int bg0 = p.prefix[b], nb = p.prefix[b + 1] - bg0;
    const float* base = p.partial + ((size_t)bg0 * p.Hq + hq) * kPartial;
    const size_t stride = (size_t)p.Hq * kPartial;
    float acc[4] = {0.f, 0.f, 0.f, 0.f}, lsum = 0.f, osum = 0.f, m_run = -INFINITY;
    for (int i0 = 4 * w; i0 < nb; i0 += 32) {   // four partials in flight per warp
        float4 v[4];
        float m[4], l[4], o[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const float* src = base + (size_t)min(i0 + u, nb - 1) * stride;
            v[u] = *reinterpret_cast<const float4*>(src + 4 * lane);
            m[u] = (i0 + u < nb) ? src[kN] : -INFINITY;
            l[u] = src[kN + 1]; o[u] = src[kN + 2];
        }
        const float m_new = fmaxf(fmaxf(fmaxf(m[0], m[1]), fmaxf(m[2], m[3])), m_run);
        if (m_new == -INFINITY) continue;
        const float keep = exp2f(m_run - m_new);
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[e] *= keep;
        lsum *= keep; osum *= keep;
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const float sc = exp2f(m[u] - m_new);   // 0 for the padding entries
            acc[0] = fmaf(v[u].x, sc, acc[0]); acc[1] = fmaf(v[u].y, sc, acc[1]);
            acc[2] = fmaf(v[u].z, sc, acc[2]); acc[3] = fmaf(v[u].w, sc, acc[3]);
            lsum = fmaf(l[u], sc, lsum);
            osum = fmaf(o[u], sc, osum);            // Eq. fold-value: + sum_t a_t o_t
        }
        m_run = m_new;
    }
    // residual window: tokens w*8 .. w*8+7, then + 64, ...
    float racc[4] = {0.f, 0.f, 0.f, 0.f}, rl = 0.f, rm = -INFINITY;
    const size_t io_row = qo_row(p, b, hq);
    int rlen = p.resid_k ? min(max(p.resid_lens[b], 0), p.resid_cap) : 0;
    rlen = max(0, rlen - row_offset(p, hq % p.G));   // an earlier query token sees fewer of the newest tokens
    if (rlen > 0) {
        const int h = hq / p.G;
        const uint2 qraw = *reinterpret_cast<const uint2*>(p.q + io_row * kN + 4 * lane);
        const float q0 = bf16_bits_to_float(qraw.x & 0xffffu), q1 = bf16_bits_to_float(qraw.x >> 16);
        const float q2 = bf16_bits_to_float(qraw.y & 0xffffu), q3 = bf16_bits_to_float(qraw.y >> 16);
        for (int t0 = 8 * w; t0 < rlen; t0 += 64) {
            uint2 kr[8], vr[8];
            float d[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const size_t off = (((size_t)b * p.resid_cap + min(t0 + u, rlen - 1)) * p.Hkv + h) * kN + 4 * lane;
                kr[u] = *reinterpret_cast<const uint2*>(p.resid_k + off);
                vr[u] = *reinterpret_cast<const uint2*>(p.resid_v + off);
            }
#pragma unroll
            for (int u = 0; u < 8; ++u)
                d[u] = fmaf(q0, bf16_bits_to_float(kr[u].x & 0xffffu),
                       fmaf(q1, bf16_bits_to_float(kr[u].x >> 16),
                       fmaf(q2, bf16_bits_to_float(kr[u].y & 0xffffu), q3 * bf16_bits_to_float(kr[u].y >> 16))));
#pragma unroll
            for (int s = 16; s >= 1; s >>= 1)
#pragma unroll
                for (int u = 0; u < 8; ++u) d[u] += __shfl_xor_sync(kFullMask, d[u], s);
            float m_new = rm;
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                d[u] = (t0 + u < rlen) ? d[u] * p.scale_log2 : -INFINITY;
                m_new = fmaxf(m_new, d[u]);
            }
            const float keep = exp2f(rm - m_new);
#pragma unroll
            for (int e = 0; e < 4; ++e) racc[e] *= keep;
            rl *= keep;
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const float pr = exp2f(d[u] - m_new);
                rl += pr;
                racc[0] = fmaf(pr, bf16_bits_to_float(vr[u].x & 0xffffu), racc[0]);
                racc[1] = fmaf(pr, bf16_bits_to_float(vr[u].x >> 16), racc[1]);
                racc[2] = fmaf(pr, bf16_bits_to_float(vr[u].y & 0xffffu), racc[2]);
                racc[3] = fmaf(pr, bf16_bits_to_float(vr[u].y >> 16), racc[3]);
            }
            rm = m_new;
        }
    }
    *reinterpret_cast<float4*>(&s_acc[w][4 * lane]) = make_float4(acc[0], acc[1], acc[2], acc[3]);
    *reinterpret_cast<float4*>(&s_racc[w][4 * lane]) = make_float4(racc[0], racc[1], racc[2], racc[3]);
    if (lane == 0) { s_mlo[w][0] = m_run; s_mlo[w][1] = lsum; s_mlo[w][2] = osum; s_mlo[w][3] = rm; s_mlo[w][4] = rl; }
    __syncthreads();
    if (w != 0) return;
    float mx = -INFINITY;
#pragma unroll
    for (int i = 0; i < 8; ++i) mx = fmaxf(mx, fmaxf(s_mlo[i][0], s_mlo[i][3]));
    acc[0] = acc[1] = acc[2] = acc[3] = 0.f;
    racc[0] = racc[1] = racc[2] = racc[3] = 0.f;
    lsum = osum = 0.f;
    if (mx != -INFINITY) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const float sc = exp2f(s_mlo[i][0] - mx), rsc = exp2f(s_mlo[i][3] - mx);
            const float4 v = *reinterpret_cast<const float4*>(&s_acc[i][4 * lane]);
            const float4 r = *reinterpret_cast<const float4*>(&s_racc[i][4 * lane]);
            acc[0] = fmaf(v.x, sc, acc[0]); acc[1] = fmaf(v.y, sc, acc[1]);
            acc[2] = fmaf(v.z, sc, acc[2]); acc[3] = fmaf(v.w, sc, acc[3]);
            racc[0] = fmaf(r.x, rsc, racc[0]); racc[1] = fmaf(r.y, rsc, racc[1]);
            racc[2] = fmaf(r.z, rsc, racc[2]); racc[3] = fmaf(r.w, rsc, racc[3]);
            lsum = fmaf(s_mlo[i][1], sc, lsum);
            lsum = fmaf(s_mlo[i][4], rsc, lsum);
            osum = fmaf(s_mlo[i][2], sc, osum);
        }
        const float inv = 1.0f / lsum;
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[e] = (acc[e] + osum) * inv;
        if (p.rotate_out) warp_fwht128(acc, lane);          // compressed part back to the unrotated domain
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[e] = fmaf(racc[e], inv, acc[e]);
    }
    if (p.out_f32)
        *reinterpret_cast<float4*>(p.out_f32 + io_row * kN + 4 * lane) = make_float4(acc[0], acc[1], acc[2], acc[3]);
    if (p.out_bf16) {
        const __nv_bfloat162 lo = __floats2bfloat162_rn(acc[0], acc[1]), hi = __floats2bfloat162_rn(acc[2], acc[3]);
        uint2 wv;
        wv.x = *reinterpret_cast<const uint32_t*>(&lo);
        wv.y = *reinterpret_cast<const uint32_t*>(&hi);
        *reinterpret_cast<uint2*>(reinterpret_cast<uint16_t*>(p.out_bf16) + io_row * kN + 4 * lane) = wv;
    }
}

// ------------------------------------------------- bf16-cache comparison baseline
//
// Plain split-K decode attention over an un-quantised bf16 cache [page][Hkv][16][128], written to be
// bound by HBM: every warp streams a contiguous token range of one (sequence, KV head) on its own --
// its own cp.async ring of 32-token K and V tiles, the query fragments, online softmax and the output
// accumulator in registers, no CTA barrier in the loop -- and leaves one partial per range.  The
// ranges ("splits") are sized on the device from the sequence lengths so that the whole cache is cut
// into about two ranges per resident warp.

#ifndef DQ_BF_WARPS
#define DQ_BF_WARPS 5
#endif
#ifndef DQ_BF_STAGES
#define DQ_BF_STAGES 2
#endif
constexpr int kBfWarps = DQ_BF_WARPS;
constexpr int kBfStages = DQ_BF_STAGES;                 // 32-token (K, V) tile pairs in flight per warp
constexpr int kBfRowStride = 272;                       // 128 bf16 + 16 bytes pad
constexpr int kBfTileBytes = kChunk * kBfRowStride;     // one 32-token K (or V) tile
constexpr int kBfWarpBytes = kBfStages * 2 * kBfTileBytes;
constexpr int kBfSmem = kBfWarps * kBfWarpBytes;
constexpr int kBfMinSplitTokens = 128;                  // a split never covers fewer tokens (bounds the partial count)

__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%0,%1,%2,%3};\n"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

__global__ void __launch_bounds__(kBfWarps * 32, 1)
dq_bf16_attention_kernel(const AttnParams p, const uint16_t* __restrict__ kp, const uint16_t* __restrict__ vp,
                         int units_target) {
    extern __shared__ __align__(128) uint8_t smem[];
    __shared__ int s_prefix[4096 + 1];   // splits before each sequence (B <= 4096)
    __shared__ long long s_tot[kBfWarps];
    pdl_launch_dependents();
    pdl_wait_prior_grid();   // the previous call's merge kernel still reads the arrays written here
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, G = p.G;
    // Every CTA sizes the splits itself (the lengths live on the device): tokens per split = a multiple of
    // 32, >= kBfMinSplitTokens, about total token-heads / units_target; then the exclusive scan of the splits
    // per sequence.  CTA 0 leaves the scan in global memory for the merge kernel.
    int split_tokens;
    {
        long long tot = 0;
        for (int b = threadIdx.x; b < p.B; b += blockDim.x) tot += min(max(p.seq_lens[b], 0), p.max_pages * DQ_PAGE_TOKENS);
#pragma unroll
        for (int d = 16; d >= 1; d >>= 1) tot += __shfl_xor_sync(kFullMask, tot, d);
        if (lane == 0) s_tot[warp] = tot;
        __syncthreads();
        tot = 0;
        for (int i = 0; i < kBfWarps; ++i) tot += s_tot[i];
        long long per = (tot * p.Hkv + units_target - 1) / units_target;
        per = max((long long)kBfMinSplitTokens, (per + kChunk - 1) / kChunk * kChunk);
        split_tokens = (int)min(per, (long long)p.max_pages * DQ_PAGE_TOKENS + kChunk);
        if (warp == 0) {
            int carry = 0;
            for (int base = 0; base < p.B; base += 32) {
                const int b = base + lane;
                int nb = 0;
                if (b < p.B) nb = (min(max(p.seq_lens[b], 0), p.max_pages * DQ_PAGE_TOKENS) + split_tokens - 1) / split_tokens;
                int incl = nb;
#pragma unroll
                for (int d = 1; d < 32; d <<= 1) {
                    const int o = __shfl_up_sync(kFullMask, incl, d);
                    if (lane >= d) incl += o;
                }
                if (b < p.B) { s_prefix[b] = carry + incl - nb; if (blockIdx.x == 0) p.prefix[b] = carry + incl - nb; }
                carry += __shfl_sync(kFullMask, incl, 31);
            }
            if (lane == 0) { s_prefix[p.B] = carry; if (blockIdx.x == 0) p.prefix[p.B] = carry; }
        }
        __syncthreads();
    }
    const uint32_t ring = smem_addr(smem) + warp * kBfWarpBytes;   // stage s: K at ring + s * 2 tiles, V one tile later
    const int units = s_prefix[p.B] * p.Hkv;
    const int g_row = lane >> 2, qd = lane & 3;
    const uint32_t frag = ((lane & 7) + (lane >> 4) * 8) * kBfRowStride + ((lane >> 3) & 1) * 16;        // K tile, B operand
    const uint32_t fragv = ((lane & 7) + ((lane >> 3) & 1) * 8) * kBfRowStride + (lane >> 4) * 16;       // V tile, transposed

    for (int u = blockIdx.x * kBfWarps + warp; u < units; u += gridDim.x * kBfWarps) {
        const int bg = u / p.Hkv, h = u - bg * p.Hkv;
        int lo = 0, hi = p.B;                     // largest b with prefix[b] <= bg
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (s_prefix[mid] <= bg) lo = mid; else hi = mid;
        }
        const int b = lo, split = bg - s_prefix[b];
        const int len = min(p.seq_lens[b], p.max_pages * DQ_PAGE_TOKENS);
        const int tok_lo = split * split_tokens, tok_hi = min(len, tok_lo + split_tokens);
        const int32_t* pt = p.page_table + (size_t)b * p.max_pages;
        __syncwarp();
        // A fragments of q for the 8 channel groups, straight from global memory: row g = lane / 4 holds head g of
        // this KV head (rows beyond G, and the upper 8 rows of the tile, are zero)
        uint32_t qa[8][2];
        {
            const uint32_t* qrow = reinterpret_cast<const uint32_t*>(p.q + ((size_t)b * p.Hq + (size_t)h * G + min(g_row, G - 1)) * kN);
#pragma unroll
            for (int cg = 0; cg < 8; ++cg) {
                qa[cg][0] = g_row < G ? qrow[cg * 8 + qd] : 0u;
                qa[cg][1] = g_row < G ? qrow[cg * 8 + 4 + qd] : 0u;
            }
        }
        auto load_chunk = [&](int tok0, int stage) {
            const uint32_t kt = ring + stage * 2 * kBfTileBytes, vt = kt + kBfTileBytes;
            const int npg = (tok0 + 16 < len) ? 2 : 1;
            for (int pg = 0; pg < npg; ++pg) {
                const size_t page = ((size_t)pt[(tok0 >> 4) + pg] * p.Hkv + h) * (size_t)(16 * kN * 2);
                const uint8_t* ks = reinterpret_cast<const uint8_t*>(kp) + page;
                const uint8_t* vs = reinterpret_cast<const uint8_t*>(vp) + page;
#pragma unroll
                for (int j = 0; j < 8; ++j) {   // 16 rows x 16 pieces of 16 bytes
                    const int i = lane + 32 * j, r = i >> 4, c = i & 15;
                    cp_async16(kt + (pg * 16 + r) * kBfRowStride + c * 16, ks + i * 16);
                    cp_async16(vt + (pg * 16 + r) * kBfRowStride + c * 16, vs + i * 16);
                }
            }
        };
        float oacc[16][4];
#pragma unroll
        for (int i = 0; i < 16; ++i) { oacc[i][0] = oacc[i][1] = oacc[i][2] = oacc[i][3] = 0.f; }
        float m_run = -INFINITY, l_run = 0.f;
#pragma unroll
        for (int s0 = 0; s0 < kBfStages - 1; ++s0) {   // prologue: the first stages - 1 chunks
            if (tok_lo + s0 * kChunk < tok_hi) load_chunk(tok_lo + s0 * kChunk, s0);
            cp_async_commit();
        }
        int stage = 0;
        for (int tok0 = tok_lo; tok0 < tok_hi; tok0 += kChunk, stage = (stage + 1 == kBfStages) ? 0 : stage + 1) {
            {
                const int ahead = tok0 + (kBfStages - 1) * kChunk;
                if (ahead < tok_hi) load_chunk(ahead, (stage + kBfStages - 1) % kBfStages);
                cp_async_commit();
            }
            cp_async_wait<kBfStages - 1>();
            __syncwarp();
            const uint32_t kt = ring + stage * 2 * kBfTileBytes, vt = kt + kBfTileBytes;
            float sacc[4][4];
#pragma unroll
            for (int i = 0; i < 4; ++i) { sacc[i][0] = sacc[i][1] = sacc[i][2] = sacc[i][3] = 0.f; }
#pragma unroll
            for (int cg = 0; cg < 8; ++cg) {
                uint32_t b0[4], b1[4];
                const uint32_t a[4] = {qa[cg][0], 0u, qa[cg][1], 0u};
                ldmatrix_x4(b0, kt + frag + cg * 32);
                ldmatrix_x4(b1, kt + frag + cg * 32 + 16 * kBfRowStride);
                mma_bf16_16816(sacc[0], a, b0[0], b0[1]);
                mma_bf16_16816(sacc[1], a, b0[2], b0[3]);
                mma_bf16_16816(sacc[2], a, b1[0], b1[1]);
                mma_bf16_16816(sacc[3], a, b1[2], b1[3]);
            }
            float mx = -INFINITY;
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int uu = 0; uu < 2; ++uu) {
                    const bool ok = tok0 + 8 * i + 2 * qd + uu < tok_hi;
                    sacc[i][uu] = ok ? sacc[i][uu] * p.scale_log2 : -INFINITY;
                    mx = fmaxf(mx, sacc[i][uu]);
                }
            mx = fmaxf(mx, __shfl_xor_sync(kFullMask, mx, 1));
            mx = fmaxf(mx, __shfl_xor_sync(kFullMask, mx, 2));
            const float m_new = fmaxf(m_run, mx);           // finite: the chunk holds at least one token of the range
            const float keep = exp2f(m_run - m_new);        // 0 on the first chunk
            m_run = m_new;
            l_run *= keep;
#pragma unroll
            for (int i = 0; i < 16; ++i) { oacc[i][0] *= keep; oacc[i][1] *= keep; }
            uint32_t pa[2][4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float p0 = exp2f(sacc[i][0] - m_new), p1 = exp2f(sacc[i][1] - m_new);
                l_run += p0 + p1;
                const __nv_bfloat162 pk = __floats2bfloat162_rn(p0, p1);
                pa[i >> 1][(i & 1) * 2] = *reinterpret_cast<const uint32_t*>(&pk);
                pa[i >> 1][(i & 1) * 2 + 1] = 0u;
            }
            // rows beyond the range end hold stale shared memory: zero weights times NaN must not
            // leak, so clear the unused V rows of the last chunk
            if (tok0 + kChunk > tok_hi) {
                for (int r = tok_hi - tok0; r < kChunk; ++r)
                    for (int c = lane; c < 64; c += 32) *reinterpret_cast<uint32_t*>(smem + (vt - smem_addr(smem)) + r * kBfRowStride + c * 4) = 0u;
                __syncwarp();
            }
#pragma unroll
            for (int cg = 0; cg < 8; ++cg) {
                uint32_t b0[4], b1[4];
                ldmatrix_x4_trans(b0, vt + fragv + cg * 32);
                ldmatrix_x4_trans(b1, vt + fragv + cg * 32 + 16 * kBfRowStride);
                mma_bf16_16816(oacc[2 * cg], pa[0], b0[0], b0[1]);
                mma_bf16_16816(oacc[2 * cg + 1], pa[0], b0[2], b0[3]);
                mma_bf16_16816(oacc[2 * cg], pa[1], b1[0], b1[1]);
                mma_bf16_16816(oacc[2 * cg + 1], pa[1], b1[2], b1[3]);
            }
            __syncwarp();   // the tiles of this stage are free for the load issued next iteration
        }
        cp_async_wait<0>();
        l_run += __shfl_xor_sync(kFullMask, l_run, 1);
        l_run += __shfl_xor_sync(kFullMask, l_run, 2);
        if (g_row < G) {
            float* dst = p.partial + ((size_t)bg * p.Hq + (size_t)h * G + g_row) * kPartial;
#pragma unroll
            for (int nt = 0; nt < 16; ++nt) *reinterpret_cast<float2*>(dst + 8 * nt + 2 * qd) = make_float2(oacc[nt][0], oacc[nt][1]);
            if (qd == 0) { dst[kN] = m_run; dst[kN + 1] = l_run; dst[kN + 2] = 0.f; }
        }
    }
}

constexpr int kMinItemTokens = 4 * kChunk;  // smallest CTA the launcher may pick (4 warps)

struct WsLayout {
    size_t off_counter, off_prefix, off_qrot, off_q16, off_qsum, off_qmu, off_partial, total;
};

inline int windows_for(int max_pages) {
    return (max_pages * DQ_PAGE_TOKENS + DQ_WINDOW_TOKENS - 1) / DQ_WINDOW_TOKENS;
}

WsLayout ws_layout(int B, int Hq, int max_pages) {
    WsLayout w;
    size_t o = 0;
    auto up = [](size_t x) { return (x + 15) & ~(size_t)15; };
    w.off_counter = o; o += 16;
    w.off_prefix = o; o += up((size_t)(B + 1) * 8);   // block prefix sums, then non-empty-sequence counts
    w.off_qrot = o; o += (size_t)B * Hq * kN * 4;
    w.off_q16 = o; o += (size_t)B * Hq * 16 * kN * 2;   // Hkv <= Hq rows blocks
    w.off_qsum = o; o += up((size_t)B * Hq * 4);
    w.off_qmu = o; o += up((size_t)B * Hq * windows_for(max_pages) * 4);
    const size_t blocks = (size_t)B * (((size_t)max_pages * DQ_PAGE_TOKENS + kMinItemTokens - 1) / kMinItemTokens);
    w.off_partial = o; o += blocks * Hq * kPartial * 4;
    w.total = o;
    return w;
}

}  // namespace

size_t dq_attn_workspace_bytes(int B, int Hq, int max_pages) { return ws_layout(B, Hq, max_pages).total; }

// Optional timing of the main kernel: CUDA events recorded on the launch stream around
// dq_attention_kernel, kept in a ring the caller drains with dq_profile_read().
namespace {
constexpr int kProfRing = 4096;
bool g_prof_on = false;
int g_prof_period = 1, g_prof_calls = 0;
int g_prof_count = 0;
cudaEvent_t g_prof_ev[kProfRing][2];
bool g_prof_made[kProfRing];
}  // namespace

void dq_attn_profile_enable(int on) {
    g_prof_on = on > 0;
    g_prof_period = on > 0 ? on : 1;   // record every on-th call
    g_prof_calls = 0;
    g_prof_count = 0;
}

int dq_attn_profile_read(float* ms, int max_records) {
    int n = 0;
    for (int i = 0; i < g_prof_count && n < max_records; ++i) {
        if (cudaEventSynchronize(g_prof_ev[i][1]) != cudaSuccess) break;
        float t = 0.f;
        if (cudaEventElapsedTime(&t, g_prof_ev[i][0], g_prof_ev[i][1]) != cudaSuccess) break;
        ms[n++] = t;
    }
    g_prof_count = 0;
    return n;
}

// SM count and opt-in shared memory of the current device, looked up once per device.
static cudaError_t device_limits(int* sm_count, int* smem_max) {
    constexpr int kDevs = 64;
    static int s_sm[kDevs], s_smem[kDevs];
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kDevs) return cudaErrorInvalidDevice;
    if (s_sm[dev] == 0) {
        int sm = 0, smem = 0;
        e = cudaDeviceGetAttribute(&sm, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return e;
        e = cudaDeviceGetAttribute(&smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
        if (e != cudaSuccess) return e;
        s_smem[dev] = smem;
        s_sm[dev] = sm;
    }
    *sm_count = s_sm[dev];
    *smem_max = s_smem[dev];
    return cudaSuccess;
}

// One pass: query tokens [q_first, q_first + q_len) of the q_total given; q_len * (Hq / Hkv) <= 8.
static cudaError_t launch_attention_pass(const DqDevTable& tk, const DqDevTable& tv, const DqAttnArgs& a, int q_total,
                                         int q_first, int q_len, cudaStream_t st) {
    int sm_count = 0, smem_max = 0;
    {
        const cudaError_t e = device_limits(&sm_count, &smem_max);
        if (e != cudaSuccess) return e;
    }
    int nw = kMaxWarps;
    const int G1 = a.Hq / a.Hkv, G = G1 * q_len;   // rows per KV head
    const bool wide = tk.hs > 1;   // token-wide streams: main kernel of dq_attention_wide.cu
    Layout L = make_layout(nw, tk.rec, tv.rec, a.B, G);
    if (wide) {
        nw = dq_attn_wide_pick_warps(tk, tv, a.B, G, smem_max);
        if (nw == 0) return cudaErrorInvalidConfiguration;
    } else {
        while (L.total > smem_max && nw > 4) {
            nw -= 2;
            L = make_layout(nw, tk.rec, tv.rec, a.B, G);
        }
        if (L.total > smem_max) return cudaErrorInvalidConfiguration;
    }

    const WsLayout w = ws_layout(a.B, a.Hq * q_len, a.max_pages);
    uint8_t* ws = static_cast<uint8_t*>(a.workspace);
    AttnParams p;
    p.q = static_cast<const uint16_t*>(a.q_bf16);
    p.k_cont = a.k_cont; p.v_cont = a.v_cont;
    p.mean_q = a.mean_q; p.mean_scale = a.mean_scale;
    p.page_table = a.page_table; p.seq_lens = a.seq_lens;
    p.counter = reinterpret_cast<int*>(ws + w.off_counter);
    p.prefix = reinterpret_cast<int*>(ws + w.off_prefix);
    p.qrot = reinterpret_cast<float*>(ws + w.off_qrot);
    p.q16 = reinterpret_cast<uint16_t*>(ws + w.off_q16);
    p.qsum = reinterpret_cast<float*>(ws + w.off_qsum);
    p.qmu = reinterpret_cast<float*>(ws + w.off_qmu);
    p.partial = reinterpret_cast<float*>(ws + w.off_partial);
    p.out_bf16 = a.out_bf16; p.out_f32 = a.out_f32;
    p.max_windows = a.max_windows; p.windows = windows_for(a.max_pages); p.max_pages = a.max_pages;
    p.B = a.B; p.Hq = a.Hq * q_len; p.Hkv = a.Hkv; p.G = G;
    p.q_len = q_len; p.G1 = G1; p.Hq1 = a.Hq;
    p.q_total = q_total; p.q_first = q_first;
    // Decode-step mode pays (dynamic item order, late wait) while the encoder's ~20 us matter: not when every
    // CTA has dozens of items anyway (upper bound from the page-table width; the lengths live on the device).
    const long long max_items = (long long)a.B * ((a.max_pages * DQ_PAGE_TOKENS + nw * kChunk - 1) / (nw * kChunk)) * a.Hkv;
    p.fused = a.fused && !wide && max_items <= 32LL * sm_count; p.attn_grid = sm_count; p.flags = p.counter;
    p.poll_limit = p.fused ? step_poll_limit() : 0;
    p.ne_before = p.prefix + (a.B + 1);
    p.item_tokens = nw * kChunk;
    p.rotate_q = tk.rotate; p.rotate_out = tv.rotate; p.has_mean = tk.has_mean;
    p.scale_log2 = a.sm_scale * 1.4426950408889634f;
    p.hkv_magic = a.Hkv > 1 ? (unsigned)((0x100000000ull + a.Hkv - 1) / a.Hkv) : 0u;
    p.hs = tk.hs; p.groups = a.Hkv / tk.hs;
    if (wide) p.hkv_magic = p.groups > 1 ? (unsigned)((0x100000000ull + p.groups - 1) / p.groups) : 0u;
    p.resid_k = static_cast<const uint16_t*>(a.resid_k); p.resid_v = static_cast<const uint16_t*>(a.resid_v);
    p.resid_lens = a.resid_lens; p.resid_cap = a.resid_cap;

    const int heads = a.B * a.Hq * q_len;
    const long long prep_warps = (long long)heads * (1 + (p.has_mean ? (p.windows + kPrepWindows - 1) / kPrepWindows : 0));
    cudaError_t e = dq_launch_pdl(dq_attn_prepare_kernel, dim3((unsigned)((prep_warps + 7) / 8)), dim3(256), 0, st, p);
    if (e != cudaSuccess) return e;
    // the four instantiations of the main kernel: decode-step mode or not, 32- or 24-bit final state
    void (*main_kernel)(DqDevTable, DqDevTable, AttnParams) =
        tk.pair ? (tk.sigma == 24 ? (p.fused ? dq_attention_kernel<true, 15, true> : dq_attention_kernel<false, 15, true>)
                                  : (p.fused ? dq_attention_kernel<true, 23, true> : dq_attention_kernel<false, 23, true>))
                : (tk.sigma == 24 ? (p.fused ? dq_attention_kernel<true, 15, false> : dq_attention_kernel<false, 15, false>)
                                  : (p.fused ? dq_attention_kernel<true, 23, false> : dq_attention_kernel<false, 23, false>));
    if (!wide) {
        e = cudaFuncSetAttribute(main_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, L.total);
        if (e != cudaSuccess) return e;
    }
    const bool prof = g_prof_on && g_prof_count < kProfRing && (g_prof_calls++ % g_prof_period) == 0;
    if (prof) {
        if (!g_prof_made[g_prof_count]) {
            if ((e = cudaEventCreate(&g_prof_ev[g_prof_count][0])) != cudaSuccess) return e;
            if ((e = cudaEventCreate(&g_prof_ev[g_prof_count][1])) != cudaSuccess) return e;
            g_prof_made[g_prof_count] = true;
        }
        cudaEventRecord(g_prof_ev[g_prof_count][0], st);
    }
    if (wide) e = dq_launch_attention_wide_main(tk, tv, p, nw, sm_count, st);
    else e = dq_launch_pdl(main_kernel, dim3(sm_count), dim3(nw * 32), (size_t)L.total, st, tk, tv, p);
    if (e != cudaSuccess) return e;
    if (prof) cudaEventRecord(g_prof_ev[g_prof_count++][1], st);
    return dq_launch_pdl(dq_attn_combine_kernel, dim3(heads), dim3(256), 0, st, p);
}

// q_len query tokens per sequence: as many passes over the cache as it takes to give every
// (query token, head) pair of a KV head one of the 8 rows of the MMA tile.
cudaError_t dq_launch_attention(const DqDevTable& tk, const DqDevTable& tv, const DqAttnArgs& a,
                                cudaStream_t st) {
    const int q_total = a.q_len > 1 ? a.q_len : 1;
    const int per_pass = DQ_MAX_GROUP / (a.Hq / a.Hkv) > 0 ? DQ_MAX_GROUP / (a.Hq / a.Hkv) : 1;
    for (int q_first = 0; q_first < q_total; q_first += per_pass) {
        const int q_len = q_total - q_first < per_pass ? q_total - q_first : per_pass;
        const cudaError_t e = launch_attention_pass(tk, tv, a, q_total, q_first, q_len, st);
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

// Decode step: the caller has just launched the step's encoder (in decode-step mode) on `st`.
cudaError_t dq_launch_step(const DqDevTable& tk, const DqDevTable& tv, const DqEncodeArgs& enc, const DqAttnArgs& a,
                           cudaStream_t st) {
    (void)enc;
    DqAttnArgs b = a;
    b.fused = 1;
    b.q_len = 1;
    return dq_launch_attention(tk, tv, b, st);
}

int* dq_attn_workspace_flags(void* workspace) { return reinterpret_cast<int*>(workspace); }

cudaError_t dq_launch_bf16_attention(const DqAttnArgs& a, const void* k_pages, const void* v_pages,
                                     cudaStream_t st) {
    const WsLayout w = ws_layout(a.B, a.Hq, a.max_pages);
    uint8_t* ws = static_cast<uint8_t*>(a.workspace);
    AttnParams p;
    p.q = static_cast<const uint16_t*>(a.q_bf16);
    p.k_cont = nullptr; p.v_cont = nullptr; p.mean_q = nullptr; p.mean_scale = nullptr;
    p.page_table = a.page_table; p.seq_lens = a.seq_lens;
    p.counter = reinterpret_cast<int*>(ws + w.off_counter);
    p.prefix = reinterpret_cast<int*>(ws + w.off_prefix);
    p.qrot = reinterpret_cast<float*>(ws + w.off_qrot);
    p.q16 = reinterpret_cast<uint16_t*>(ws + w.off_q16);
    p.qsum = reinterpret_cast<float*>(ws + w.off_qsum);
    p.qmu = reinterpret_cast<float*>(ws + w.off_qmu);
    p.partial = reinterpret_cast<float*>(ws + w.off_partial);
    p.out_bf16 = a.out_bf16; p.out_f32 = nullptr;
    p.max_windows = 0; p.windows = 0; p.has_mean = 0; p.max_pages = a.max_pages;
    p.B = a.B; p.Hq = a.Hq; p.Hkv = a.Hkv; p.G = a.Hq / a.Hkv;
    p.item_tokens = kBfMinSplitTokens;
    p.rotate_q = 0; p.rotate_out = 0;
    p.scale_log2 = a.sm_scale * 1.4426950408889634f;
    p.hkv_magic = 0;
    p.hs = 1; p.groups = a.Hkv;
    p.q_len = 1; p.G1 = p.G; p.Hq1 = a.Hq; p.q_total = 1; p.q_first = 0;
    p.fused = 0; p.attn_grid = 0; p.poll_limit = 0; p.flags = p.counter; p.ne_before = p.prefix + (a.B + 1);
    p.resid_k = nullptr; p.resid_v = nullptr; p.resid_lens = nullptr; p.resid_cap = 0;
    const int heads = a.B * a.Hq;
    int sm_count = 0, smem_max = 0;
    cudaError_t e = device_limits(&sm_count, &smem_max);
    if (e != cudaSuccess) return e;
    if (kBfSmem + 17 * 1024 > smem_max) return cudaErrorInvalidConfiguration;   // ring + the static scan arrays
    e = cudaFuncSetAttribute(dq_bf16_attention_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kBfSmem);
    if (e != cudaSuccess) return e;
    e = dq_launch_pdl(dq_bf16_attention_kernel, dim3(sm_count), dim3(kBfWarps * 32), (size_t)kBfSmem, st, p,
                      static_cast<const uint16_t*>(k_pages), static_cast<const uint16_t*>(v_pages),
                      2 * sm_count * kBfWarps);
    if (e != cudaSuccess) return e;
    return dq_launch_pdl(dq_attn_combine_kernel, dim3(heads), dim3(256), 0, st, p);
}

// ------------------------------------------------ attention without any allocation
//
// Scratch for dq_decode_attention_static: a fixed array in device global memory that exists
// in every CUDA context which loads this library, from load until the context ends.  Host
// code may not use the symbol `g_static_scratch` as a pointer (on the host it is only a
// stand-in for the device object); its device address is looked up once per device with
// cudaGetSymbolAddress and that address is what the kernels receive.
static __device__ __align__(256) unsigned char g_static_scratch[DQ_STATIC_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
void* g_static_scratch_addr[kMaxDevices];
bool g_static_scratch_known[kMaxDevices];
}  // namespace

// Device address of the static scratch array on the current device (looked up on first use).
cudaError_t dq_attn_static_scratch(void** out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    if (!g_static_scratch_known[dev]) {
        void* addr = nullptr;
        e = cudaGetSymbolAddress(&addr, g_static_scratch);
        if (e != cudaSuccess) return e;
        g_static_scratch_addr[dev] = addr;
        g_static_scratch_known[dev] = true;
    }
    *out = g_static_scratch_addr[dev];
    return cudaSuccess;
}

// Same launches as dq_launch_attention, with the event-recording measurement aid held off so
// that nothing on this route can create a CUDA object.
cudaError_t dq_launch_attention_static(const DqDevTable& tk, const DqDevTable& tv, const DqAttnArgs& a,
                                       cudaStream_t st) {
    const bool was_on = g_prof_on;
    g_prof_on = false;
    const cudaError_t e = dq_launch_attention(tk, tv, a, st);
    g_prof_on = was_on;
    return e;
}
