// Fused decode-step attention over rANS-coded KV containers (Sec. 4.5 "Decoding";
// Algorithm 2; Appendix A Eq. fold-key / fold-value) for sm_100a.
//
// Launch sequence per call (one stream):
//   dq_attn_prepare_kernel   rotate q (q' = H q / sqrt(128)), per-sequence block prefix
//                            sums, reset of the work counter
//   dq_attention_kernel      persistent, one CTA per SM; CTAs pull work items
//                            (sequence, KV head, block of NW*32 tokens) from an atomic
//                            counter.  Each warp owns 32 tokens of the item: lane l runs the
//                            rANS state machines of token l (K stream, then V stream) out of
//                            shared memory, levels go to a small fp16 tile and from there
//                            into mma.sync contractions against q' (K) and the softmax
//                            weights (V).  s, o and the window mean are applied after the
//                            contraction.  The next item's records are prefetched with
//                            cp.async while the current one is decoded.
//   dq_attn_combine_kernel   log-sum-exp merge of the per-block partials, inverse rotation
//                            of the output when V was rotated, bf16 / f32 store.
//
// q' and the softmax weights enter the tensor cores as fp16 hi + lo pairs (rows g and g + 8
// of the 16-row operand), so the contraction carries ~22 mantissa bits; levels 0..15 are
// exact in fp16.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "dq_device.cuh"
#include "dq_internal.h"

using namespace dqdev;

namespace {

constexpr int kN = DQ_HEAD_DIM;
constexpr int kChunk = 32;             // tokens per warp per item
constexpr uint32_t kL = 1u << 23;
constexpr int kTileStride = 48;        // bytes per token row of a [32 tok][16 ch] fp16 tile (+16 pad)
constexpr int kTileBytes = kChunk * kTileStride;
constexpr int kQ16Stride = 272;        // bytes per row of the fp16 q' operand (128 halves + pad)
constexpr int kPartial = 132;          // floats per partial record: 128 acc, m, l, 2 pad
constexpr int kMergeStride = 136;      // floats per (slot, head) row of the merge buffer
constexpr int kMaxWarps = 16;
constexpr int kMaxPerThread = DQ_MAX_GROUP * kN / 128;  // merge outputs per thread at 4 warps

struct Item {
    int b, h, blk, len, bg, valid, pad0, pad1;
};

struct Layout {
    int stage_k, stage_v, stage_bytes;  // per warp per buffer
    int off_lutk, off_lutv, off_prefix, off_qf32, off_q16, off_qsum, off_item, off_red, off_stage,
        off_tiles, total;
    int warp_tile_bytes;
};

__host__ __device__ inline int align16(int x) { return (x + 15) & ~15; }

__host__ __device__ inline Layout make_layout(int nw, int rec_k, int rec_v, int B) {
    Layout L;
    L.stage_k = align16(kChunk * rec_k);
    L.stage_v = align16(kChunk * rec_v);
    L.stage_bytes = L.stage_k + L.stage_v + kN + 16;  // + INT8 mean row + its scale
    L.warp_tile_bytes = 2 * kTileBytes + kChunk * 16;  // K tile, V tile, per-token (sK,oK,sV,oV)
    int o = 0;
    L.off_lutk = o; o += 256 * 32 * 4;
    L.off_lutv = o; o += 256 * 32 * 4;
    L.off_prefix = o; o += align16((B + 1) * 4);
    L.off_qf32 = o; o += 2 * DQ_MAX_GROUP * kN * 4;
    L.off_q16 = o; o += 16 * kQ16Stride;
    L.off_qsum = o; o += DQ_MAX_GROUP * 4;
    L.off_item = o; o += 2 * (int)sizeof(Item);
    L.off_red = o; o += 3 * kMaxWarps * DQ_MAX_GROUP * 4;
    L.off_stage = o; o += 2 * nw * L.stage_bytes;
    L.off_tiles = o; o += nw * L.warp_tile_bytes;
    L.total = o + 256;  // slack: a malformed record may be over-read by up to 136 + 8 bytes
    return L;
}

struct AttnParams {
    const uint16_t* q;
    const uint8_t* k_cont;
    const uint8_t* v_cont;
    const int8_t* mean_q;
    const float* mean_scale;
    const int32_t* page_table;
    const int32_t* seq_lens;
    int* counter;
    int* prefix;      // [B + 1] blocks before sequence b
    float* qrot;      // [B][Hq][128]
    float* partial;   // [blocks][Hq][kPartial]
    void* out_bf16;
    float* out_f32;
    int max_windows, max_pages, B, Hq, Hkv, G, item_tokens, rotate_q, rotate_out;
    float scale_log2;  // sm_scale * log2(e)
};

// ------------------------------------------------------------------ prepare

__global__ void __launch_bounds__(256)
dq_attn_prepare_kernel(AttnParams p) {
    const int lane = threadIdx.x & 31;
    const int wid = blockIdx.x * 8 + (threadIdx.x >> 5);
    if (wid < p.B * p.Hq) {
        const uint2 raw = *reinterpret_cast<const uint2*>(p.q + (size_t)wid * kN + 4 * lane);
        float v[4] = {bf16_bits_to_float(raw.x & 0xffffu), bf16_bits_to_float(raw.x >> 16),
                      bf16_bits_to_float(raw.y & 0xffffu), bf16_bits_to_float(raw.y >> 16)};
        if (p.rotate_q) warp_fwht128(v, lane);
        *reinterpret_cast<float4*>(p.qrot + (size_t)wid * kN + 4 * lane) = make_float4(v[0], v[1], v[2], v[3]);
    }
    if (blockIdx.x == 0 && threadIdx.x < 32) {  // exclusive scan of blocks per sequence
        int carry = 0;
        for (int base = 0; base < p.B; base += 32) {
            const int b = base + lane;
            int nb = 0;
            if (b < p.B) nb = (min(max(p.seq_lens[b], 0), p.max_pages * DQ_PAGE_TOKENS) + p.item_tokens - 1) / p.item_tokens;
            int incl = nb;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const int o = __shfl_up_sync(kFullMask, incl, d);
                if (lane >= d) incl += o;
            }
            if (b < p.B) p.prefix[b] = carry + incl - nb;
            carry += __shfl_sync(kFullMask, incl, 31);
        }
        if (lane == 0) { p.prefix[p.B] = carry; *p.counter = 0; }
    }
}

// --------------------------------------------------------------------- main

// Decode 16 symbols of one stream (Algorithm 2) and pack their levels as 8 fp16x2 words.
// x: rANS state; ptr: shared-memory byte address of the next renormalisation byte;
// lut: shared address of this lane's column of the 32-way replicated table (entry z at
// lut + z * 128).  Renormalisation bytes come from a 4-byte window refreshed every 4 symbols
// (a symbol consumes at most one byte).
__device__ __forceinline__ void decode16(uint32_t& x, uint32_t& ptr, uint32_t lut, uint32_t (&packed)[8]) {
#pragma unroll
    for (int q4 = 0; q4 < 4; ++q4) {
        const uint32_t win = lds32_unaligned(ptr);
        uint32_t sel = 0x2104u;
        uint32_t e[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            e[i] = lds32(lut + ((x & 255u) << 7));
            x = ((e[i] >> 8) & 255u) * (x >> 8) + (e[i] & 255u);
            if (x < kL) { x = __byte_perm(x, win, sel); sel += 1u; }
        }
        ptr += sel - 0x2104u;
        packed[2 * q4] = __byte_perm(e[0], e[1], 0x7632u);
        packed[2 * q4 + 1] = __byte_perm(e[2], e[3], 0x7632u);
    }
}

__device__ __forceinline__ uint32_t pack_half2(float a, float b) {
    const __half2 h = __floats2half2_rn(a, b);
    return *reinterpret_cast<const uint32_t*>(&h);
}

__global__ void __launch_bounds__(kMaxWarps * 32, 1)
dq_attention_kernel(const __grid_constant__ DqDevTable TK, const __grid_constant__ DqDevTable TV,
                    const AttnParams p) {
    extern __shared__ __align__(128) uint8_t smem[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nthreads = blockDim.x, nw = nthreads >> 5;
    const int G = p.G;
    const Layout L = make_layout(nw, TK.rec, TV.rec, p.B);
    const uint32_t sbase = smem_addr(smem);

    uint32_t* lutk = reinterpret_cast<uint32_t*>(smem + L.off_lutk);
    uint32_t* lutv = reinterpret_cast<uint32_t*>(smem + L.off_lutv);
    int* prefix = reinterpret_cast<int*>(smem + L.off_prefix);
    float* qf32 = reinterpret_cast<float*>(smem + L.off_qf32);
    float* qsum = reinterpret_cast<float*>(smem + L.off_qsum);
    Item* items = reinterpret_cast<Item*>(smem + L.off_item);
    float* red_m = reinterpret_cast<float*>(smem + L.off_red);
    float* red_l = red_m + kMaxWarps * DQ_MAX_GROUP;
    float* red_o = red_l + kMaxWarps * DQ_MAX_GROUP;
    float* mbuf = reinterpret_cast<float*>(smem + L.off_tiles);  // aliases the tiles between items

    for (int i = tid; i < 256 * 32; i += nthreads) {
        lutk[i] = TK.lut[i >> 5];
        lutv[i] = TV.lut[i >> 5];
    }
    for (int i = tid; i <= p.B; i += nthreads) prefix[i] = p.prefix[i];
    __syncthreads();
    const int total_items = prefix[p.B] * p.Hkv;

    const uint32_t my_lutk = sbase + L.off_lutk + lane * 4, my_lutv = sbase + L.off_lutv + lane * 4;
    const uint32_t my_tiles = sbase + L.off_tiles + warp * L.warp_tile_bytes;
    const uint32_t ktile = my_tiles, vtile = my_tiles + kTileBytes, scal = my_tiles + 2 * kTileBytes;
    const int merge_slots = (nw * L.warp_tile_bytes) / (G * kMergeStride * 4);

    auto fetch_item = [&](int buf) {  // thread 0 only
        Item it;
        it.valid = 0; it.b = it.h = it.blk = it.len = it.bg = 0; it.pad0 = it.pad1 = 0;
        const int idx = atomicAdd(p.counter, 1);
        if (idx < total_items) {
            it.valid = 1;
            it.h = idx % p.Hkv;
            it.bg = idx / p.Hkv;
            int lo = 0, hi = p.B;
            while (hi - lo > 1) {
                const int mid = (lo + hi) >> 1;
                if (prefix[mid] <= it.bg) lo = mid; else hi = mid;
            }
            it.b = lo;
            it.blk = it.bg - prefix[lo];
            it.len = min(p.seq_lens[lo], p.max_pages * DQ_PAGE_TOKENS);
        }
        items[buf] = it;
    };

    auto issue_loads = [&](int buf) {
        const Item it = items[buf];
        if (it.valid) {
            const uint32_t stage = sbase + L.off_stage + (buf * nw + warp) * L.stage_bytes;
            const int tok0 = (it.blk * nw + warp) * kChunk;
            if (tok0 < it.len) {
                const int32_t* pt = p.page_table + (size_t)it.b * p.max_pages + (tok0 >> 4);
                const int npg = (tok0 + 16 < it.len) ? 2 : 1;
                for (int pg = 0; pg < npg; ++pg) {
                    const size_t page = (size_t)pt[pg] * p.Hkv + it.h;
                    const uint8_t* ks = p.k_cont + page * (size_t)(16 * TK.rec);
                    const uint8_t* vs = p.v_cont + page * (size_t)(16 * TV.rec);
                    for (int i = lane; i < TK.rec; i += 32) cp_async16(stage + pg * 16 * TK.rec + i * 16, ks + i * 16);
                    for (int i = lane; i < TV.rec; i += 32)
                        cp_async16(stage + L.stage_k + pg * 16 * TV.rec + i * 16, vs + i * 16);
                }
                if (TK.has_mean) {
                    const size_t mi = ((size_t)it.b * p.max_windows + tok0 / DQ_WINDOW_TOKENS) * p.Hkv + it.h;
                    if (lane < 8) cp_async16(stage + L.stage_k + L.stage_v + lane * 16, p.mean_q + mi * kN + lane * 16);
                    if (lane == 8) cp_async4(stage + L.stage_k + L.stage_v + kN, p.mean_scale + mi);
                }
            }
            for (int i = tid; i < G * 32; i += nthreads)  // q' rows of this KV head's group
                cp_async16(sbase + L.off_qf32 + buf * (DQ_MAX_GROUP * kN * 4) + i * 16,
                           p.qrot + ((size_t)it.b * p.Hq + (size_t)it.h * G) * kN + i * 4);
        }
        cp_async_commit();
    };

    int buf = 0;
    if (tid == 0) fetch_item(0);
    __syncthreads();
    issue_loads(0);

    const int g_row = lane >> 2, qd = lane & 3;

    while (true) {
        const Item it = items[buf];
        if (!it.valid) break;
        if (tid == 0) fetch_item(buf ^ 1);
        __syncthreads();
        issue_loads(buf ^ 1);
        cp_async_wait<1>();
        __syncthreads();

        // fp16 hi/lo operand of q' (rows g: hi, rows 8 + g: lo) and row sums
        {
            const float* qf = qf32 + buf * (DQ_MAX_GROUP * kN);
            for (int i = tid; i < 8 * kN; i += nthreads) {
                const int g = i >> 7, ch = i & (kN - 1);
                float v = (g < G) ? qf[g * kN + ch] : 0.f;
                const __half hi = __float2half_rn(v);
                const __half lo = __float2half_rn(v - __half2float(hi));
                *reinterpret_cast<__half*>(smem + L.off_q16 + g * kQ16Stride + ch * 2) = hi;
                *reinterpret_cast<__half*>(smem + L.off_q16 + (g + 8) * kQ16Stride + ch * 2) = lo;
            }
            for (int g = warp; g < DQ_MAX_GROUP; g += nw) {
                float s = 0.f;
                if (g < G) {
                    const float4 v = *reinterpret_cast<const float4*>(qf + g * kN + 4 * lane);
                    s = (v.x + v.y) + (v.z + v.w);
                }
#pragma unroll
                for (int d = 16; d >= 1; d >>= 1) s += __shfl_xor_sync(kFullMask, s, d);
                if (lane == 0) qsum[g] = s;
            }
        }
        __syncthreads();

        // ------------------------------------------------ this warp's 32 tokens
        float oacc[16][4];
#pragma unroll
        for (int i = 0; i < 16; ++i) { oacc[i][0] = oacc[i][1] = oacc[i][2] = oacc[i][3] = 0.f; }
        float m_run = -INFINITY, l_run = 0.f, off_run = 0.f;

        const int tok0 = (it.blk * nw + warp) * kChunk;
        if (tok0 < it.len) {
            const uint32_t stage = sbase + L.off_stage + (buf * nw + warp) * L.stage_bytes;
            const uint32_t rk = stage + lane * TK.rec, rv = stage + L.stage_k + lane * TV.rec;
            const uint32_t hk = lds32_unaligned(rk), hv = lds32_unaligned(rv);
            uint32_t xk = lds32_unaligned(rk + 4), xv = lds32_unaligned(rv + 4);
            {
                const float sK = __half2float(__ushort_as_half((unsigned short)(hk & 0xffffu)));
                const float oK = __half2float(__ushort_as_half((unsigned short)(hk >> 16)));
                const float sV = __half2float(__ushort_as_half((unsigned short)(hv & 0xffffu)));
                const float oV = __half2float(__ushort_as_half((unsigned short)(hv >> 16)));
                asm volatile("st.shared.v4.f32 [%0], {%1,%2,%3,%4};\n" ::"r"(scal + lane * 16), "f"(sK), "f"(oK),
                             "f"(sV), "f"(oV) : "memory");
            }
            // q' . mean of this chunk's window, for the head row this thread owns
            float qmu = 0.f;
            if (TK.has_mean) {
                const uint32_t mrow = stage + L.stage_k + L.stage_v;
                const uint32_t q4 = lds32(mrow + lane * 4);
                const float msc = __uint_as_float(lds32(mrow + kN));
                float mu[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) mu[e] = msc * (float)(int)(int8_t)((q4 >> (8 * e)) & 0xffu);
                const float* qf = qf32 + buf * (DQ_MAX_GROUP * kN);
                for (int g = 0; g < G; ++g) {
                    const float4 v = *reinterpret_cast<const float4*>(qf + g * kN + 4 * lane);
                    float s = v.x * mu[0] + v.y * mu[1] + v.z * mu[2] + v.w * mu[3];
#pragma unroll
                    for (int d = 16; d >= 1; d >>= 1) s += __shfl_xor_sync(kFullMask, s, d);
                    if (g == g_row) qmu = s;
                }
            }
            const float qs = (g_row < G) ? qsum[g_row] : 0.f;

            // ---- keys: S[g][t] = sum_j q'_gj level_tj  (Eq. fold-key, inner sum)
            float sacc[4][4];
#pragma unroll
            for (int i = 0; i < 4; ++i) { sacc[i][0] = sacc[i][1] = sacc[i][2] = sacc[i][3] = 0.f; }
            {
                uint32_t ptr = rk + 8;
                const uint32_t a_addr = sbase + L.off_q16 + ((lane & 7) + ((lane >> 3) & 1) * 8) * kQ16Stride +
                                        (lane >> 4) * 16;
                const uint32_t b_addr = ktile + ((lane & 7) + (lane >> 4) * 8) * kTileStride + ((lane >> 3) & 1) * 16;
#pragma unroll 1
                for (int cg = 0; cg < 8; ++cg) {
                    uint32_t pk[8];
                    decode16(xk, ptr, my_lutk, pk);
                    asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};\n" ::"r"(ktile + lane * kTileStride),
                                 "r"(pk[0]), "r"(pk[1]), "r"(pk[2]), "r"(pk[3]) : "memory");
                    asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};\n" ::"r"(ktile + lane * kTileStride + 16),
                                 "r"(pk[4]), "r"(pk[5]), "r"(pk[6]), "r"(pk[7]) : "memory");
                    __syncwarp();
                    uint32_t a[4], b0[4], b1[4];
                    ldmatrix_x4(a, a_addr + cg * 32);
                    ldmatrix_x4(b0, b_addr);
                    ldmatrix_x4(b1, b_addr + 16 * kTileStride);
                    mma_f16_16816(sacc[0], a, b0[0], b0[1]);
                    mma_f16_16816(sacc[1], a, b0[2], b0[3]);
                    mma_f16_16816(sacc[2], a, b1[0], b1[1]);
                    mma_f16_16816(sacc[3], a, b1[2], b1[3]);
                    __syncwarp();
                }
            }

            // ---- affine terms, softmax weights (base 2), fp16 hi/lo A operands for P.V
            uint32_t pa[2][4];
            {
                float lg[4][2], sv_t[4][2], ov_t[4][2];
                float mx = -INFINITY;
#pragma unroll
                for (int i = 0; i < 4; ++i)
#pragma unroll
                    for (int u = 0; u < 2; ++u) {
                        const int tk = 8 * i + 2 * qd + u;
                        float4 m4;
                        asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];\n"
                                     : "=f"(m4.x), "=f"(m4.y), "=f"(m4.z), "=f"(m4.w) : "r"(scal + tk * 16));
                        const float S = sacc[i][u] + sacc[i][2 + u];
                        const bool ok = tok0 + tk < it.len;
                        lg[i][u] = ok ? p.scale_log2 * fmaf(m4.x, S, fmaf(m4.y, qs, qmu)) : -INFINITY;
                        sv_t[i][u] = ok ? m4.z : 0.f;
                        ov_t[i][u] = ok ? m4.w : 0.f;
                        mx = fmaxf(mx, lg[i][u]);
                    }
                mx = fmaxf(mx, __shfl_xor_sync(kFullMask, mx, 1));
                mx = fmaxf(mx, __shfl_xor_sync(kFullMask, mx, 2));
                m_run = mx;
                const float m_use = (mx == -INFINITY) ? 0.f : mx;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    float hi[2], lo[2];
#pragma unroll
                    for (int u = 0; u < 2; ++u) {
                        const float pr = exp2f(lg[i][u] - m_use);
                        l_run += pr;
                        off_run = fmaf(pr, ov_t[i][u], off_run);
                        const float ps = pr * sv_t[i][u];
                        hi[u] = __half2float(__float2half_rn(ps));
                        lo[u] = ps - hi[u];
                    }
                    pa[i >> 1][(i & 1) * 2 + 0] = pack_half2(hi[0], hi[1]);
                    pa[i >> 1][(i & 1) * 2 + 1] = pack_half2(lo[0], lo[1]);
                }
            }

            // ---- values: O[g][j] += sum_t (a_t s_t) level_tj  (Eq. fold-value, first sum)
            {
                uint32_t ptr = rv + 8;
                const uint32_t b_addr = vtile + ((lane & 7) + ((lane >> 3) & 1) * 8) * kTileStride + (lane >> 4) * 16;
#pragma unroll
                for (int cg = 0; cg < 8; ++cg) {
                    uint32_t pk[8];
                    decode16(xv, ptr, my_lutv, pk);
                    asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};\n" ::"r"(vtile + lane * kTileStride),
                                 "r"(pk[0]), "r"(pk[1]), "r"(pk[2]), "r"(pk[3]) : "memory");
                    asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};\n" ::"r"(vtile + lane * kTileStride + 16),
                                 "r"(pk[4]), "r"(pk[5]), "r"(pk[6]), "r"(pk[7]) : "memory");
                    __syncwarp();
                    uint32_t b0[4], b1[4];
                    ldmatrix_x4_trans(b0, b_addr);                      // tokens 0..15
                    ldmatrix_x4_trans(b1, b_addr + 16 * kTileStride);   // tokens 16..31
                    mma_f16_16816(oacc[2 * cg], pa[0], b0[0], b0[1]);
                    mma_f16_16816(oacc[2 * cg + 1], pa[0], b0[2], b0[3]);
                    mma_f16_16816(oacc[2 * cg], pa[1], b1[0], b1[1]);
                    mma_f16_16816(oacc[2 * cg + 1], pa[1], b1[2], b1[3]);
                    __syncwarp();
                }
            }
        }

        // ------------------------------------------------ merge the warps of this item
        l_run += __shfl_xor_sync(kFullMask, l_run, 1);
        l_run += __shfl_xor_sync(kFullMask, l_run, 2);
        off_run += __shfl_xor_sync(kFullMask, off_run, 1);
        off_run += __shfl_xor_sync(kFullMask, off_run, 2);
        if (qd == 0) {
            red_m[warp * DQ_MAX_GROUP + g_row] = m_run;
            red_l[warp * DQ_MAX_GROUP + g_row] = l_run;
            red_o[warp * DQ_MAX_GROUP + g_row] = off_run;
        }
        __syncthreads();  // also: every warp is done with its tiles -> merge buffer may alias them
        float m_all = -INFINITY;
        for (int w = 0; w < nw; ++w) m_all = fmaxf(m_all, red_m[w * DQ_MAX_GROUP + g_row]);
        const float m_base = (m_all == -INFINITY) ? 0.f : m_all;
        const float my_scale = exp2f(m_run - m_base);

        // output slot of this thread: (head og, channel oc) and (og + G/.., ...) handled below
        float tot[kMaxPerThread];
#pragma unroll
        for (int r = 0; r < kMaxPerThread; ++r) tot[r] = 0.f;
        for (int w0 = 0; w0 < nw; w0 += merge_slots) {
            if (warp >= w0 && warp < w0 + merge_slots && g_row < G) {
                float* dst = mbuf + ((warp - w0) * G + g_row) * kMergeStride + 2 * qd;
#pragma unroll
                for (int nt = 0; nt < 16; ++nt) {
                    const float2 v = make_float2((oacc[nt][0] + oacc[nt][2]) * my_scale,
                                                 (oacc[nt][1] + oacc[nt][3]) * my_scale);
                    *reinterpret_cast<float2*>(dst + 8 * nt) = v;
                }
            }
            __syncthreads();
            const int cnt = min(merge_slots, nw - w0);
#pragma unroll
            for (int r = 0; r < kMaxPerThread; ++r) {
                const int e = tid + r * nthreads;
                if (e < G * kN) {
                    const int g = e >> 7, ch = e & (kN - 1);
                    float s = 0.f;
                    for (int w = 0; w < cnt; ++w) s += mbuf[(w * G + g) * kMergeStride + ch];
                    tot[r] += s;
                }
            }
            __syncthreads();
        }
#pragma unroll
        for (int r = 0; r < kMaxPerThread; ++r) {
            const int e = tid + r * nthreads;
            if (e >= G * kN) break;
            const int g = e >> 7, ch = e & (kN - 1);
            float mg = -INFINITY;
            for (int w = 0; w < nw; ++w) mg = fmaxf(mg, red_m[w * DQ_MAX_GROUP + g]);
            const float mb = (mg == -INFINITY) ? 0.f : mg;
            float lsum = 0.f, osum = 0.f;
            for (int w = 0; w < nw; ++w) {
                const float sc = exp2f(red_m[w * DQ_MAX_GROUP + g] - mb);
                lsum = fmaf(red_l[w * DQ_MAX_GROUP + g], sc, lsum);
                osum = fmaf(red_o[w * DQ_MAX_GROUP + g], sc, osum);
            }
            float* dst = p.partial + ((size_t)it.bg * p.Hq + (size_t)it.h * G + g) * kPartial;
            dst[ch] = tot[r] + osum;               // Eq. fold-value: + sum_t a_t o_t
            if (ch == 0) { dst[kN] = mg; dst[kN + 1] = lsum; }
        }
        __syncthreads();
        buf ^= 1;
    }
    cp_async_wait<0>();
}

// ------------------------------------------------------------------ combine

__global__ void __launch_bounds__(256)
dq_attn_combine_kernel(AttnParams p) {
    const int lane = threadIdx.x & 31;
    const int wid = blockIdx.x * 8 + (threadIdx.x >> 5);
    if (wid >= p.B * p.Hq) return;
    const int b = wid / p.Hq, hq = wid % p.Hq;
    const int bg0 = p.prefix[b], nb = p.prefix[b + 1] - bg0;
    float mx = -INFINITY;
    for (int i = 0; i < nb; ++i) mx = fmaxf(mx, p.partial[((size_t)(bg0 + i) * p.Hq + hq) * kPartial + kN]);
    float acc[4] = {0.f, 0.f, 0.f, 0.f}, lsum = 0.f;
    if (mx != -INFINITY) {
        for (int i = 0; i < nb; ++i) {
            const float* src = p.partial + ((size_t)(bg0 + i) * p.Hq + hq) * kPartial;
            const float sc = exp2f(src[kN] - mx);
            const float4 v = *reinterpret_cast<const float4*>(src + 4 * lane);
            acc[0] = fmaf(v.x, sc, acc[0]); acc[1] = fmaf(v.y, sc, acc[1]);
            acc[2] = fmaf(v.z, sc, acc[2]); acc[3] = fmaf(v.w, sc, acc[3]);
            lsum = fmaf(src[kN + 1], sc, lsum);
        }
        const float inv = 1.0f / lsum;
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[e] *= inv;
        if (p.rotate_out) warp_fwht128(acc, lane);
    }
    if (p.out_f32)
        *reinterpret_cast<float4*>(p.out_f32 + (size_t)wid * kN + 4 * lane) = make_float4(acc[0], acc[1], acc[2], acc[3]);
    if (p.out_bf16) {
        const __nv_bfloat162 lo = __floats2bfloat162_rn(acc[0], acc[1]), hi = __floats2bfloat162_rn(acc[2], acc[3]);
        uint2 w;
        w.x = *reinterpret_cast<const uint32_t*>(&lo);
        w.y = *reinterpret_cast<const uint32_t*>(&hi);
        *reinterpret_cast<uint2*>(reinterpret_cast<uint16_t*>(p.out_bf16) + (size_t)wid * kN + 4 * lane) = w;
    }
}

// ------------------------------------------------- bf16-cache comparison baseline

constexpr int kBfWarps = 4;
constexpr int kBfRowStride = 272;                       // 128 bf16 + 16 bytes pad
constexpr int kBfTileBytes = kChunk * kBfRowStride;     // one warp's K (or V) tile
constexpr int kBfSmem = 16 * kBfRowStride + kBfWarps * 2 * kBfTileBytes + 3 * kBfWarps * 8 * 4 +
                        kBfWarps * 8 * kMergeStride * 4;

__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%0,%1,%2,%3};\n"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// Plain split-K decode attention over an un-quantised bf16 cache [page][Hkv][16][128].
// One CTA per (block of 128 tokens, KV head, sequence); each warp owns 32 tokens.
__global__ void __launch_bounds__(kBfWarps * 32)
dq_bf16_attention_kernel(const AttnParams p, const uint16_t* __restrict__ kp, const uint16_t* __restrict__ vp) {
    extern __shared__ __align__(128) uint8_t smem[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int b = blockIdx.z, h = blockIdx.y, blk = blockIdx.x, G = p.G;
    const int bg0 = p.prefix[b];
    if (blk >= p.prefix[b + 1] - bg0) return;
    const int len = min(p.seq_lens[b], p.max_pages * DQ_PAGE_TOKENS);
    const uint32_t sbase = smem_addr(smem);
    const uint32_t q16 = sbase;
    const uint32_t kt = sbase + 16 * kBfRowStride + warp * 2 * kBfTileBytes, vt = kt + kBfTileBytes;
    float* red_m = reinterpret_cast<float*>(smem + 16 * kBfRowStride + kBfWarps * 2 * kBfTileBytes);
    float* red_l = red_m + kBfWarps * 8;
    float* mbuf = red_l + 2 * kBfWarps * 8;

    const int tok0 = (blk * kBfWarps + warp) * kChunk;
    if (tok0 < len) {
        const int npg = (tok0 + 16 < len) ? 2 : 1;
        for (int pg = 0; pg < npg; ++pg) {
            const size_t page = (size_t)p.page_table[(size_t)b * p.max_pages + (tok0 >> 4) + pg] * p.Hkv + h;
            const uint8_t* ks = reinterpret_cast<const uint8_t*>(kp) + page * (16 * kN * 2);
            const uint8_t* vs = reinterpret_cast<const uint8_t*>(vp) + page * (16 * kN * 2);
            for (int i = lane; i < 256; i += 32) {   // 16 rows x 16 chunks of 16 bytes
                const int r = i >> 4, c = i & 15;
                cp_async16(kt + (pg * 16 + r) * kBfRowStride + c * 16, ks + i * 16);
                cp_async16(vt + (pg * 16 + r) * kBfRowStride + c * 16, vs + i * 16);
            }
        }
    }
    cp_async_commit();
    for (int i = tid; i < 16 * 64; i += blockDim.x) {   // q rows (bf16 pairs), zero beyond G
        const int g = i >> 6, c = i & 63;
        uint32_t v = 0;
        if (g < G) v = *reinterpret_cast<const uint32_t*>(p.q + ((size_t)b * p.Hq + (size_t)h * G + g) * kN + 2 * c);
        *reinterpret_cast<uint32_t*>(smem + g * kBfRowStride + c * 4) = v;
    }
    cp_async_wait<0>();
    __syncthreads();

    const int g_row = lane >> 2, qd = lane & 3;
    float oacc[16][4];
#pragma unroll
    for (int i = 0; i < 16; ++i) { oacc[i][0] = oacc[i][1] = oacc[i][2] = oacc[i][3] = 0.f; }
    float m_run = -INFINITY, l_run = 0.f;
    if (tok0 < len) {
        float sacc[4][4];
#pragma unroll
        for (int i = 0; i < 4; ++i) { sacc[i][0] = sacc[i][1] = sacc[i][2] = sacc[i][3] = 0.f; }
        const uint32_t a_addr = q16 + ((lane & 7) + ((lane >> 3) & 1) * 8) * kBfRowStride + (lane >> 4) * 16;
        const uint32_t b_addr = kt + ((lane & 7) + (lane >> 4) * 8) * kBfRowStride + ((lane >> 3) & 1) * 16;
#pragma unroll
        for (int cg = 0; cg < 8; ++cg) {
            uint32_t a[4], b0[4], b1[4];
            ldmatrix_x4(a, a_addr + cg * 32);
            ldmatrix_x4(b0, b_addr + cg * 32);
            ldmatrix_x4(b1, b_addr + cg * 32 + 16 * kBfRowStride);
            mma_bf16_16816(sacc[0], a, b0[0], b0[1]);
            mma_bf16_16816(sacc[1], a, b0[2], b0[3]);
            mma_bf16_16816(sacc[2], a, b1[0], b1[1]);
            mma_bf16_16816(sacc[3], a, b1[2], b1[3]);
        }
        float mx = -INFINITY;
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                const bool ok = tok0 + 8 * i + 2 * qd + u < len;
                sacc[i][u] = ok ? sacc[i][u] * p.scale_log2 : -INFINITY;
                mx = fmaxf(mx, sacc[i][u]);
            }
        mx = fmaxf(mx, __shfl_xor_sync(kFullMask, mx, 1));
        mx = fmaxf(mx, __shfl_xor_sync(kFullMask, mx, 2));
        m_run = mx;
        const float m_use = (mx == -INFINITY) ? 0.f : mx;
        uint32_t pa[2][4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float p0 = exp2f(sacc[i][0] - m_use), p1 = exp2f(sacc[i][1] - m_use);
            l_run += p0 + p1;
            const __nv_bfloat162 pk = __floats2bfloat162_rn(p0, p1);
            pa[i >> 1][(i & 1) * 2] = *reinterpret_cast<const uint32_t*>(&pk);
            pa[i >> 1][(i & 1) * 2 + 1] = 0u;
        }
        // rows beyond the sequence end hold stale shared memory: zero weights times NaN must not
        // leak, so clear the unused V rows of the last chunk
        if (tok0 + kChunk > len) {
            for (int r = len - tok0; r < kChunk; ++r)
                for (int c = lane; c < 64; c += 32) *reinterpret_cast<uint32_t*>(smem + (vt - sbase) + r * kBfRowStride + c * 4) = 0u;
            __syncwarp();
        }
        const uint32_t v_addr = vt + ((lane & 7) + ((lane >> 3) & 1) * 8) * kBfRowStride + (lane >> 4) * 16;
#pragma unroll
        for (int cg = 0; cg < 8; ++cg) {
            uint32_t b0[4], b1[4];
            ldmatrix_x4_trans(b0, v_addr + cg * 32);
            ldmatrix_x4_trans(b1, v_addr + cg * 32 + 16 * kBfRowStride);
            mma_bf16_16816(oacc[2 * cg], pa[0], b0[0], b0[1]);
            mma_bf16_16816(oacc[2 * cg + 1], pa[0], b0[2], b0[3]);
            mma_bf16_16816(oacc[2 * cg], pa[1], b1[0], b1[1]);
            mma_bf16_16816(oacc[2 * cg + 1], pa[1], b1[2], b1[3]);
        }
    }
    l_run += __shfl_xor_sync(kFullMask, l_run, 1);
    l_run += __shfl_xor_sync(kFullMask, l_run, 2);
    if (qd == 0) { red_m[warp * 8 + g_row] = m_run; red_l[warp * 8 + g_row] = l_run; }
    __syncthreads();
    float m_all = -INFINITY;
    for (int w = 0; w < kBfWarps; ++w) m_all = fmaxf(m_all, red_m[w * 8 + g_row]);
    const float my_scale = exp2f(m_run - ((m_all == -INFINITY) ? 0.f : m_all));
    if (g_row < G) {
        float* dst = mbuf + (warp * G + g_row) * kMergeStride + 2 * qd;
#pragma unroll
        for (int nt = 0; nt < 16; ++nt)
            *reinterpret_cast<float2*>(dst + 8 * nt) = make_float2(oacc[nt][0] * my_scale, oacc[nt][1] * my_scale);
    }
    __syncthreads();
    for (int e = tid; e < G * kN; e += blockDim.x) {
        const int g = e >> 7, ch = e & (kN - 1);
        float mg = -INFINITY, s = 0.f, lsum = 0.f;
        for (int w = 0; w < kBfWarps; ++w) mg = fmaxf(mg, red_m[w * 8 + g]);
        const float mb = (mg == -INFINITY) ? 0.f : mg;
        for (int w = 0; w < kBfWarps; ++w) {
            s += mbuf[(w * G + g) * kMergeStride + ch];
            lsum = fmaf(red_l[w * 8 + g], exp2f(red_m[w * 8 + g] - mb), lsum);
        }
        float* dst = p.partial + ((size_t)(bg0 + blk) * p.Hq + (size_t)h * G + g) * kPartial;
        dst[ch] = s;
        if (ch == 0) { dst[kN] = mg; dst[kN + 1] = lsum; }
    }
}

constexpr int kMinItemTokens = 4 * kChunk;  // smallest CTA the launcher may pick (4 warps)

struct WsLayout {
    size_t off_counter, off_prefix, off_qrot, off_partial, total;
};

WsLayout ws_layout(int B, int Hq, int max_pages) {
    WsLayout w;
    size_t o = 0;
    w.off_counter = o; o += 16;
    w.off_prefix = o; o += ((size_t)(B + 1) * 4 + 15) & ~(size_t)15;
    w.off_qrot = o; o += (size_t)B * Hq * kN * 4;
    const size_t blocks = (size_t)B * (((size_t)max_pages * DQ_PAGE_TOKENS + kMinItemTokens - 1) / kMinItemTokens);
    w.off_partial = o; o += blocks * Hq * kPartial * 4;
    w.total = o;
    return w;
}

}  // namespace

size_t dq_attn_workspace_bytes(int B, int Hq, int max_pages) { return ws_layout(B, Hq, max_pages).total; }

cudaError_t dq_launch_attention(const DqDevTable& tk, const DqDevTable& tv, const DqAttnArgs& a,
                                cudaStream_t st) {
    static int sm_count = 0, smem_max = 0;
    if (sm_count == 0) {
        int dev = 0;
        cudaError_t e = cudaGetDevice(&dev);
        if (e != cudaSuccess) return e;
        e = cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return e;
        e = cudaDeviceGetAttribute(&smem_max, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
        if (e != cudaSuccess) return e;
    }
    int nw = kMaxWarps;
    Layout L = make_layout(nw, tk.rec, tv.rec, a.B);
    while (L.total > smem_max && nw > 4) {
        nw -= 4;
        L = make_layout(nw, tk.rec, tv.rec, a.B);
    }
    if (L.total > smem_max) return cudaErrorInvalidConfiguration;

    const WsLayout w = ws_layout(a.B, a.Hq, a.max_pages);
    uint8_t* ws = static_cast<uint8_t*>(a.workspace);
    AttnParams p;
    p.q = static_cast<const uint16_t*>(a.q_bf16);
    p.k_cont = a.k_cont; p.v_cont = a.v_cont;
    p.mean_q = a.mean_q; p.mean_scale = a.mean_scale;
    p.page_table = a.page_table; p.seq_lens = a.seq_lens;
    p.counter = reinterpret_cast<int*>(ws + w.off_counter);
    p.prefix = reinterpret_cast<int*>(ws + w.off_prefix);
    p.qrot = reinterpret_cast<float*>(ws + w.off_qrot);
    p.partial = reinterpret_cast<float*>(ws + w.off_partial);
    p.out_bf16 = a.out_bf16; p.out_f32 = a.out_f32;
    p.max_windows = a.max_windows; p.max_pages = a.max_pages;
    p.B = a.B; p.Hq = a.Hq; p.Hkv = a.Hkv; p.G = a.Hq / a.Hkv;
    p.item_tokens = nw * kChunk;
    p.rotate_q = tk.rotate; p.rotate_out = tv.rotate;
    p.scale_log2 = a.sm_scale * 1.4426950408889634f;

    const int heads = a.B * a.Hq;
    dq_attn_prepare_kernel<<<(heads + 7) / 8, 256, 0, st>>>(p);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(dq_attention_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, L.total);
    if (e != cudaSuccess) return e;
    dq_attention_kernel<<<sm_count, nw * 32, L.total, st>>>(tk, tv, p);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    dq_attn_combine_kernel<<<(heads + 7) / 8, 256, 0, st>>>(p);
    return cudaGetLastError();
}

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
    p.partial = reinterpret_cast<float*>(ws + w.off_partial);
    p.out_bf16 = a.out_bf16; p.out_f32 = nullptr;
    p.max_windows = 0; p.max_pages = a.max_pages;
    p.B = a.B; p.Hq = a.Hq; p.Hkv = a.Hkv; p.G = a.Hq / a.Hkv;
    p.item_tokens = kBfWarps * kChunk;
    p.rotate_q = 0; p.rotate_out = 0;
    p.scale_log2 = a.sm_scale * 1.4426950408889634f;
    const int heads = a.B * a.Hq;
    dq_attn_prepare_kernel<<<(heads + 7) / 8, 256, 0, st>>>(p);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(dq_bf16_attention_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kBfSmem);
    if (e != cudaSuccess) return e;
    const int max_blocks = (a.max_pages * DQ_PAGE_TOKENS + p.item_tokens - 1) / p.item_tokens;
    dq_bf16_attention_kernel<<<dim3(max_blocks, a.Hkv, a.B), kBfWarps * 32, kBfSmem, st>>>(
        p, static_cast<const uint16_t*>(k_pages), static_cast<const uint16_t*>(v_pages));
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    dq_attn_combine_kernel<<<(heads + 7) / 8, 256, 0, st>>>(p);
    return cudaGetLastError();
}
