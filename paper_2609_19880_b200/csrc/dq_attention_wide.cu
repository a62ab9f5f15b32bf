// Fused decode-step attention over token-wide rANS streams (Sec. 5.1 "Implementation
// details": each token is one group of hs * 128 values; Sec. 4.5 "Decoding": a stream is
// decoded once, one KV head at a time, and feeds that head's attention directly).
//
// Same machinery as the per-head kernel (lane = token, levels -> fp16 tile -> mma.sync,
// affine terms after the contraction, K of step s interleaved with V of step s - 1, static
// round-robin items), with these differences:
//   * a work item is (sequence, stream group, block of NW * 32 tokens); it takes hs steps, one
//     per head of the group, and the rANS state of a token runs on across the steps;
//   * a record (335 / 235 bytes at the paper's setting) is far too large to stage whole: each
//     warp keeps a ring of record words per tensor kind in shared memory, [row][lane] with
//     row = word index mod ROWS.  Records are stored word-interleaved per page, so one ring
//     row of a warp is two contiguous 64-byte runs of global memory (16-byte cp.async pieces,
//     coalesced), and lane l reads only bank l (no conflicts whatever the lanes' positions).
//     Before every 16-symbol tile the warp extends the ring to (largest word index of its
//     lanes) + 10 rows, which covers the 36 bytes two tiles can consume; a lane that lags more
//     than ROWS - 10 words behind the fastest lane reads its words from global memory
//     instead (correct, slower; K streams that do not fill their container lag by up to
//     ~90 bytes, hence 32 rows for K and 16 for V, which always fill theirs).
#include "dq_attention_common.cuh"

using namespace dqdev;
using namespace dqattn;

namespace {

constexpr int kRowsK = 32, kRowsV = 16;        // ring rows (4-byte words per lane)
constexpr int kRingK = kRowsK * 128, kRingV = kRowsV * 128;
constexpr int kTile = 1024;                    // [32 tok][16 ch] fp16, 32-byte rows, halves swizzled by (row >> 2) & 1
constexpr int kFillRows = 12;                  // rows fetched when a stream starts (header + 40 bytes)
constexpr int kAhead = 10;                     // rows kept beyond the fastest lane's word index
constexpr int kWideWarps = 15;                 // most warps per CTA: the rings of a 16th do not fit the shared memory

struct Item {
    int b, grp, blk, len, bg, valid;
};

// Shared-memory layout.  Everything the decode loop touches sits at a compile-time offset from
// the CTA's base or from the warp's own region, so the addresses cost no registers.
constexpr int kOffLutK = 0, kOffLutV = kOffLutK + 256 * 32 * 4;
constexpr int kOffQ16 = kOffLutV + 256 * 32 * 4;                       // [2] fp16 q' operand
constexpr int kOffQsum = kOffQ16 + 2 * kQ16Bytes;                      // [2][8] sum of q'
constexpr int kOffRed = kOffQsum + 2 * DQ_MAX_GROUP * 4;               // [warp][head] maxima, [2][head] step maxima
constexpr int kOffPages = kOffRed + (kMaxWarps + 2) * DQ_MAX_GROUP * 4;   // per warp: page ids of 4 items in flight
constexpr int kOffPrevRow = kOffPages + kMaxWarps * 4 * 2 * 4;         // [2] partial row of the pending V step
constexpr int kOffWarp = (kOffPrevRow + 16 + 127) & ~127;              // per-warp regions
constexpr int kWRingK = 0, kWRingV = kWRingK + kRingK, kWTileK = kWRingV + kRingV, kWTileV = kWTileK + kTile;
constexpr int kWQmu = kWTileV + kTile;                                 // [2][8] q'.mean of the warp's window
constexpr int kWObuf = kWQmu + 2 * DQ_MAX_GROUP * 4;                   // [G][kORow] output slot

__host__ __device__ inline int warp_stride(int G) { return kWObuf + G * kORow * 4; }
__host__ __device__ inline int align16w(int x) { return (x + 15) & ~15; }
// total bytes: fixed part, nw warp regions, then the per-sequence block prefix sums and lengths
__host__ __device__ inline int wide_smem_bytes(int nw, int B, int G) {
    return kOffWarp + nw * warp_stride(G) + align16w((2 * B + 1) * 4);
}

// Decode 16 symbols of one stream (Algorithm 2) out of the warp's ring and pack their levels as
// 8 fp16x2 words.  ptr is the index of the next renormalisation byte within the record; the
// 4-byte window is reloaded every 4 symbols from ring rows (ptr >> 2) and (ptr >> 2) + 1.
template <int ROWS>
__device__ __forceinline__ void decode16_ring(uint32_t& x, uint32_t& ptr, uint32_t ring_lane, uint32_t lut, uint32_t one,
                                              uint32_t (&packed)[8]) {
    constexpr uint32_t kMask = (uint32_t)(ROWS - 1) << 7;
#pragma unroll
    for (int q4 = 0; q4 < 4; ++q4) {
        const uint32_t t = ptr << 5;   // (word index) * 128 + junk below bit 7
        const uint32_t lo = lds32(ring_lane + (t & kMask));
        const uint32_t hi = lds32(ring_lane + ((t + 128u) & kMask));
        const uint32_t win = __funnelshift_r(lo, hi, ptr << 3);
        uint32_t sel = 0x2104u;
        uint32_t e[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            e[i] = lds32(dp4a_u32(x, 0x80u, lut));
            const uint32_t f = dp4a_u32(e[i], 0x01000000u, 0u);
            const uint32_t tt = f * (x >> 8);
            x = dp4a_u32(e[i], 1u, tt);
            asm("{.reg .pred p; setp.lt.u32 p, %0, 0x800000; @p prmt.b32 %0, %0, %2, %1; "
                "@p mad.lo.u32 %1, %3, %3, %1;}"
                : "+r"(x), "+r"(sel) : "r"(win), "r"(one));
        }
        ptr += sel - 0x2104u;
        packed[2 * q4] = __byte_perm(e[0], e[1], 0x6521u);
        packed[2 * q4 + 1] = __byte_perm(e[2], e[3], 0x6521u);
    }
}

// Paired-symbol tables: one step decodes the levels of two consecutive channels, 8 steps the 16; an entry is
// code(b) << 24 | f << 16 | code(a) << 8 | (z - c), code(m) the high byte of fp16(m), so the step's fp16x2 word is
// the entry with its f and (z - c) bytes cleared.
template <int ROWS>
__device__ __forceinline__ void decode16_ring_pairs(uint32_t& x, uint32_t& ptr, uint32_t ring_lane, uint32_t lut, uint32_t one,
                                                    uint32_t (&packed)[8]) {
    constexpr uint32_t kMask = (uint32_t)(ROWS - 1) << 7;
#pragma unroll
    for (int q4 = 0; q4 < 2; ++q4) {
        const uint32_t t = ptr << 5;
        const uint32_t lo = lds32(ring_lane + (t & kMask));
        const uint32_t hi = lds32(ring_lane + ((t + 128u) & kMask));
        const uint32_t win = __funnelshift_r(lo, hi, ptr << 3);
        uint32_t sel = 0x2104u;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint32_t e = lds32(dp4a_u32(x, 0x80u, lut));
            const uint32_t f = dp4a_u32(e, 0x00010000u, 0u);
            const uint32_t tt = f * (x >> 8);
            x = dp4a_u32(e, 1u, tt);
            asm("{.reg .pred p; setp.lt.u32 p, %0, 0x800000; @p prmt.b32 %0, %0, %2, %1; "
                "@p mad.lo.u32 %1, %3, %3, %1;}"
                : "+r"(x), "+r"(sel) : "r"(win), "r"(one));
            packed[4 * q4 + i] = e & 0xff00ff00u;
        }
        ptr += sel - 0x2104u;
    }
}

// The same 16 symbols for a warp in which some lane lags too far behind the ring: such a lane
// (`fast` false) takes its window words from the record in global memory (col: its word 0;
// consecutive words are 16 words apart).  Rare, kept out of line.
struct Decoded16 {
    uint32_t packed[8];
    uint32_t x, ptr;
};
__device__ __noinline__ Decoded16 decode16_mixed(uint32_t x, uint32_t ptr, uint32_t ring_lane, uint32_t ring_mask,
                                                 uint32_t lut, bool fast, const uint32_t* col, int rec_words, bool pairs) {
    Decoded16 r;
    for (int q4 = 0; q4 < (pairs ? 2 : 4); ++q4) {
        const uint32_t t = ptr << 5;
        uint32_t lo, hi;
        if (fast) {
            lo = lds32(ring_lane + (t & ring_mask));
            hi = lds32(ring_lane + ((t + 128u) & ring_mask));
        } else {
            const int wi = min((int)(ptr >> 2), rec_words - 2);
            lo = __ldg(col + (size_t)wi * 16);
            hi = __ldg(col + (size_t)wi * 16 + 16);
        }
        uint32_t win = __funnelshift_r(lo, hi, ptr << 3);
        uint32_t e[4];
        for (int i = 0; i < 4; ++i) {
            e[i] = lds32(lut + ((x & 255u) << 7));
            x = (pairs ? (e[i] >> 16) & 255u : e[i] >> 24) * (x >> 8) + (e[i] & 255u);
            if (x < (1u << 23)) {   // at most one byte per symbol
                x = (x << 8) | (win & 255u);
                win >>= 8;
                ++ptr;
            }
        }
        if (pairs) {
            for (int i = 0; i < 4; ++i) r.packed[4 * q4 + i] = e[i] & 0xff00ff00u;
        } else {
            r.packed[2 * q4] = __byte_perm(e[0], e[1], 0x6521u);
            r.packed[2 * q4 + 1] = __byte_perm(e[2], e[3], 0x6521u);
        }
    }
    r.x = x; r.ptr = ptr;
    return r;
}

// State of one tensor kind's streams in a warp.
struct Chain {
    uint32_t x, ptr;        // rANS state, next byte index within the record (per lane)
    uint32_t E;             // ring holds rows [.., E) (warp-uniform)
    uint32_t src16;         // per lane: source of its 16-byte piece of row 0, in 16-byte units from the container base
    bool active;            // lane's token exists
    bool copy_ok;           // lane's piece belongs to a page that holds tokens of the sequence
};

// Extend the ring to kAhead rows beyond the fastest lane (call with all earlier copies landed
// and the warp converged); returns whether this lane may read the ring during the next tile.
// A tile consumes at most 16 bytes, so at most 5 rows (40 pieces, two per lane) are due.
template <int ROWS>
__device__ __forceinline__ bool ring_advance(Chain& c, uint32_t ring_piece, const uint8_t* cont, int rec_words, int lane) {
    const uint32_t wi = c.ptr >> 2;
    const uint32_t wmax = __reduce_max_sync(kFullMask, c.active ? wi : 0u);
    const uint32_t Enew = max(c.E, min(wmax + (uint32_t)kAhead, (uint32_t)rec_words));
    uint32_t row = c.E + (uint32_t)(lane >> 3);
    if (row < Enew && c.copy_ok)
        cp_async16(ring_piece + ((row & (ROWS - 1)) << 7), cont + (size_t)(c.src16 + row * 4u) * 16);
    row += 4;
    if (row < Enew && c.copy_ok)
        cp_async16(ring_piece + ((row & (ROWS - 1)) << 7), cont + (size_t)(c.src16 + row * 4u) * 16);
    c.E = Enew;
    return !c.active || (wi + ROWS >= Enew);
}

// Word 0 of this lane's own record (global): the container block of its page starts at 64 times
// the src16 / 4 of the lane whose piece lies in that page (lane 0 or 4).
__device__ __forceinline__ const uint32_t* own_column(const Chain& c, const uint8_t* cont, int lane) {
    const uint32_t blk64 = __shfl_sync(kFullMask, c.src16, (lane >> 4) * 4) >> 2;
    return reinterpret_cast<const uint32_t*>(cont + (size_t)blk64 * 64) + (lane & 15);
}

// One step: 128 channels (one head), 16 at a time; K streams of the current step's head and V
// streams of the previous step's head decoded in one instruction stream (as in the per-head
// kernel), each out of its ring.
template <bool DO_K, bool DO_V, bool PAIRS>
__device__ __forceinline__ void wide_pass(Chain& ck, Chain& cv, uint32_t ringk, uint32_t ringv, const uint8_t* k_cont,
                                          const uint8_t* v_cont, int rwk, int rwv, uint32_t lutk, uint32_t lutv,
                                          uint32_t one, uint32_t ktile, uint32_t vtile, uint32_t q16, uint32_t obuf,
                                          int lane, int G, float (&sacc)[4][4], const uint32_t (&pb_hi)[2][2],
                                          const uint32_t (&pb_lo)[2][2]) {
    const uint32_t a_addr = q16 + ((lane & 7) + ((lane >> 3) & 1) * 8) * kQ16Stride + (lane >> 4) * 16;
    // tile rows are 32 bytes; the 16-byte half h of row r sits at half h ^ ((r >> 2) & 1)
    const int lrow = (lane & 7) + (lane >> 4) * 8;
    const uint32_t ld_off = lrow * 32 + ((((lane >> 3) & 1) ^ ((lrow >> 2) & 1)) << 4);
    const uint32_t st_lo = lane * 32 + (((lane >> 2) & 1) << 4), st_hi = lane * 32 + ((((lane >> 2) & 1) ^ 1) << 4);
    const uint32_t o_addr = obuf + ((2 * (lane & 3)) * kORow + (lane >> 2)) * 4;
    const uint32_t ringk_lane = ringk + lane * 4, ringv_lane = ringv + lane * 4;
    const uint32_t ringk_piece = ringk + ((lane & 7) << 4), ringv_piece = ringv + ((lane & 7) << 4);
#pragma unroll 1
    for (int cg = 0; cg < 8; ++cg) {
        cp_async_wait<0>();
        __syncwarp();
        bool fk = true, fv = true;
        if (DO_K) fk = ring_advance<kRowsK>(ck, ringk_piece, k_cont, rwk, lane);
        if (DO_V) fv = ring_advance<kRowsV>(cv, ringv_piece, v_cont, rwv, lane);
        cp_async_commit();
        uint32_t pk[8], pv[8];
        if (__all_sync(kFullMask, fk && fv)) {
            if (DO_K) { if (PAIRS) decode16_ring_pairs<kRowsK>(ck.x, ck.ptr, ringk_lane, lutk, one, pk); else decode16_ring<kRowsK>(ck.x, ck.ptr, ringk_lane, lutk, one, pk); }
            if (DO_V) { if (PAIRS) decode16_ring_pairs<kRowsV>(cv.x, cv.ptr, ringv_lane, lutv, one, pv); else decode16_ring<kRowsV>(cv.x, cv.ptr, ringv_lane, lutv, one, pv); }
        } else {   // some lane lags behind its ring: that lane reads global memory (rare, out of line)
            if (DO_K) {
                const Decoded16 r = decode16_mixed(ck.x, ck.ptr, ringk_lane, (uint32_t)(kRowsK - 1) << 7, lutk, fk,
                                                   own_column(ck, k_cont, lane), rwk, PAIRS);
#pragma unroll
                for (int i = 0; i < 8; ++i) pk[i] = r.packed[i];
                ck.x = r.x; ck.ptr = r.ptr;
            }
            if (DO_V) {
                const Decoded16 r = decode16_mixed(cv.x, cv.ptr, ringv_lane, (uint32_t)(kRowsV - 1) << 7, lutv, fv,
                                                   own_column(cv, v_cont, lane), rwv, PAIRS);
#pragma unroll
                for (int i = 0; i < 8; ++i) pv[i] = r.packed[i];
                cv.x = r.x; cv.ptr = r.ptr;
            }
        }
        if (DO_K) { sts128(ktile + st_lo, pk); sts128(ktile + st_hi, pk + 4); }
        if (DO_V) { sts128(vtile + st_lo, pv); sts128(vtile + st_hi, pv + 4); }
        __syncwarp();
        if (DO_K) {
            uint32_t a[4], b0[4], b1[4];
            ldmatrix_x4(a, a_addr + cg * 32);
            ldmatrix_x4(b0, ktile + ld_off);
            ldmatrix_x4(b1, ktile + ld_off + 16 * 32);
            mma_f16_16816(sacc[0], a, b0[0], b0[1]);
            mma_f16_16816(sacc[1], a, b0[2], b0[3]);
            mma_f16_16816(sacc[2], a, b1[0], b1[1]);
            mma_f16_16816(sacc[3], a, b1[2], b1[3]);
        }
        if (DO_V) {
            uint32_t a0[4], a1[4];
            float o[4] = {0.f, 0.f, 0.f, 0.f};
            ldmatrix_x4_trans(a0, vtile + ld_off);
            ldmatrix_x4_trans(a1, vtile + ld_off + 16 * 32);
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

template <bool PAIRS>
__global__ void __launch_bounds__(kWideWarps * 32, 1)
dq_attention_wide_kernel(const __grid_constant__ DqDevTable TK, const __grid_constant__ DqDevTable TV,
                         const AttnParams p) {
    extern __shared__ __align__(128) uint8_t smem[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nthreads = blockDim.x, nw = nthreads >> 5;
    const int G = p.G, hs = p.hs, groups = p.groups;
    const int rwk = TK.rec_words, rwv = TV.rec_words;
    const uint32_t sbase = smem_addr(smem);
    const int wstride = warp_stride(G);

    uint32_t* lutk = reinterpret_cast<uint32_t*>(smem + kOffLutK);
    uint32_t* lutv = reinterpret_cast<uint32_t*>(smem + kOffLutV);
    int* prefix = reinterpret_cast<int*>(smem + kOffWarp + nw * wstride);
    int* s_len = prefix + (p.B + 1);
    float* qsum = reinterpret_cast<float*>(smem + kOffQsum);        // [2][8]
    float* red_m = reinterpret_cast<float*>(smem + kOffRed);        // [warp][head] chunk maxima
    float* red_M = red_m + kMaxWarps * DQ_MAX_GROUP;                // [2][head] step maxima

    pdl_launch_dependents();
    for (int i = tid; i < 256 * 32; i += nthreads) {
        lutk[i] = TK.lut[i >> 5];
        lutv[i] = TV.lut[i >> 5];
    }
    pdl_wait_prior_grid();
    for (int i = tid; i <= p.B; i += nthreads) {
        prefix[i] = p.prefix[i];
        if (i < p.B) s_len[i] = min(p.seq_lens[i], p.max_pages * DQ_PAGE_TOKENS);
    }
    __syncthreads();
    const int total_items = prefix[p.B] * groups;

    const uint32_t my_lutk = sbase + kOffLutK + lane * 4, my_lutv = sbase + kOffLutV + lane * 4;
    const uint32_t wb = sbase + kOffWarp + warp * wstride;   // this warp's region
    const uint32_t ringk = wb + kWRingK, ringv = wb + kWRingV, ktile = wb + kWTileK, vtile = wb + kWTileV;
    const uint32_t my_obuf = wb + kWObuf, my_qmu = wb + kWQmu;
    const uint32_t one = (sbase >> 31) | 1u;
    const int g_row = lane >> 2, qd = lane & 3;

    auto item_of = [&](int n, int hint) {
        Item it;
        it.valid = 0; it.b = hint; it.grp = it.blk = it.len = it.bg = 0;
        const unsigned idx = blockIdx.x + (unsigned)n * gridDim.x;
        if (idx < (unsigned)total_items) {
            it.valid = 1;
            it.bg = p.hkv_magic ? (int)__umulhi(idx, p.hkv_magic) : (int)idx;   // idx / groups
            it.grp = (int)(idx - (unsigned)it.bg * (unsigned)groups);
            int b = hint;
            while (prefix[b + 1] <= it.bg) ++b;
            it.b = b;
            it.blk = it.bg - prefix[b];
            it.len = s_len[b];
        }
        return it;
    };
    int* my_pages = reinterpret_cast<int*>(smem + kOffPages) + warp * 8;
    long long* s_prev_row = reinterpret_cast<long long*>(smem + kOffPrevRow);
    auto fetch_pages = [&](int n, const Item& it) {
        const int tok0 = (it.blk * nw + warp) * kChunk;
        if (it.valid && tok0 < it.len && lane < 2 && tok0 + 16 * lane < it.len)
            cp_async4(smem_addr(my_pages + (n & 3) * 2 + lane),
                      p.page_table + (size_t)it.b * p.max_pages + (tok0 >> 4) + lane);
    };
    // q' operand, sum of q' and q'.mean of this warp's window for (item, head): what a step's
    // contraction and logits need; double-buffered by step parity
    auto issue_step_loads = [&](int s, const Item& it, int k) {
        if (!it.valid) return;
        const int h = it.grp * hs + k;
        const uint16_t* qsrc = p.q16 + ((size_t)it.b * p.Hkv + h) * 16 * kN;
        for (int i = tid; i < 16 * 16; i += nthreads)
            cp_async16(sbase + kOffQ16 + (s & 1) * kQ16Bytes + (i >> 4) * kQ16Stride + (i & 15) * 16, qsrc + i * 8);
        if (tid < G)
            cp_async4(sbase + kOffQsum + ((s & 1) * DQ_MAX_GROUP + tid) * 4, p.qsum + (size_t)it.b * p.Hq + (size_t)h * G + tid);
        const int tok0 = (it.blk * nw + warp) * kChunk;
        if (p.has_mean && tok0 < it.len && lane < G)
            cp_async4(my_qmu + ((s & 1) * DQ_MAX_GROUP + lane) * 4,
                      p.qmu + ((size_t)it.b * p.Hq + (size_t)h * G + lane) * p.windows + tok0 / DQ_WINDOW_TOKENS);
    };
    // Start the streams of item `it` (slot n mod 4 of the page ids) for one tensor kind:
    // per-lane sources and the first rows of the ring.  The caller has made sure nobody still
    // reads the ring.
    auto start_chain = [&](Chain& c, int n, const Item& it, const uint8_t* cont, int rec_words, uint32_t ring, int rows) {
        const int tok0 = (it.blk * nw + warp) * kChunk;
        c.active = it.valid && tok0 + lane < it.len;
        const int pslot = (lane >> 2) & 1;     // page of this lane's 16-byte piece (tokens 4 (lane & 7) ..)
        c.copy_ok = it.valid && tok0 + 16 * pslot < it.len;
        c.src16 = 0u;
        if (c.copy_ok) {
            const unsigned pg = (unsigned)my_pages[(n & 3) * 2 + pslot];
            c.src16 = (pg * (unsigned)groups + (unsigned)it.grp) * (unsigned)rec_words * 4u + (unsigned)(lane & 3);
        }
        const int fill = min(kFillRows, rec_words);
        if (c.copy_ok)
            for (int j = lane; j < fill * 8; j += 32) {
                const uint32_t row = (uint32_t)(j >> 3);
                cp_async16(ring + ((row & (uint32_t)(rows - 1)) << 7) + ((lane & 7) << 4), cont + (size_t)(c.src16 + row * 4u) * 16);
            }
        c.E = (uint32_t)fill;
        c.ptr = 8u;
    };

    Chain ck, cv;
    ck.x = cv.x = 1u << 23; ck.ptr = cv.ptr = 8u; ck.E = cv.E = 0u; ck.src16 = cv.src16 = 0u;
    ck.active = cv.active = false; ck.copy_ok = cv.copy_ok = false;

    // prologue: page ids of items 0 and 1, K ring and step loads of (item 0, head 0)
    int hint = 0;
    Item cur = item_of(0, 0);
    {
        fetch_pages(0, cur);
        fetch_pages(1, item_of(1, cur.b));
        cp_async_commit();
        cp_async_wait<0>();
        __syncwarp();
        start_chain(ck, 0, cur, p.k_cont, rwk, ringk, kRowsK);
        issue_step_loads(0, cur, 0);
        cp_async_commit();
        hint = cur.b;
    }

    int nK = 0, kK = 0;                // K chain: item index of this CTA, head within the group
    bool have_prev = false;            // a V step is pending (the previous step had a K step)
    int kV = 0;                        // head of the pending V step
    bool wv = false;                   // this warp holds tokens of the pending V step's item
    int nwv = 0;                       // warps that hold tokens of that item
    uint32_t hk = 0u, hv = 0u;        // headers (s, o as fp16 pairs) of the K item's tokens
    uint32_t pb_hi[2][2] = {{0u, 0u}, {0u, 0u}}, pb_lo[2][2] = {{0u, 0u}, {0u, 0u}};

    for (int s = 0;; ++s) {
        if (!cur.valid && !have_prev) break;
        cp_async_wait<0>();
        __syncthreads();   // operand of this step visible; last step's merge reads are done

        // next step's descriptor: same item, next head -- or the next item's first head
        const bool last_head = (kK == hs - 1);
        Item nxt = cur;
        if (last_head) nxt = item_of(nK + 1, cur.b);
        if (cur.valid) {
            issue_step_loads(s + 1, nxt, last_head ? 0 : kK + 1);
            if (kK == 0) fetch_pages(nK + 2, item_of(nK + 2, item_of(nK + 1, cur.b).b));
        }
        cp_async_commit();

        // streams that start with this step
        if (have_prev && kV == 0)            // V streams of the pending item: state from ring row 1 (fetched after the last pass)
            cv.x = lds32(ringv + 128 + lane * 4);
        int tok0 = (cur.blk * nw + warp) * kChunk;
        if (cur.valid && kK == 0) {          // K streams of `cur`: header and state from ring rows 0, 1
            hk = lds32(ringk + lane * 4);
            ck.x = lds32(ringk + 128 + lane * 4);
            if (ck.active) {                  // V header of the same tokens: needed for this item's weights
                const size_t pg = (size_t)my_pages[(nK & 3) * 2 + (lane >> 4)];
                const uint32_t* vcol = reinterpret_cast<const uint32_t*>(p.v_cont + (pg * groups + cur.grp) * ((size_t)rwv * 64)) + (lane & 15);
                hv = __ldg(vcol);
            }
        }

        const uint32_t q16 = sbase + kOffQ16 + (s & 1) * kQ16Bytes;
        float sacc[4][4];
#pragma unroll
        for (int i = 0; i < 4; ++i) { sacc[i][0] = sacc[i][1] = sacc[i][2] = sacc[i][3] = 0.f; }
        // a warp whose 32 tokens lie beyond the sequence end skips the decode (its logits are masked,
        // its output slot is left out of the merge)
        bool wk = cur.valid && tok0 < cur.len;
        if (wk && wv)
            wide_pass<true, true, PAIRS>(ck, cv, ringk, ringv, p.k_cont, p.v_cont, rwk, rwv, my_lutk, my_lutv, one, ktile, vtile, q16,
                                  my_obuf, lane, G, sacc, pb_hi, pb_lo);
        else if (wk)
            wide_pass<true, false, PAIRS>(ck, cv, ringk, ringv, p.k_cont, p.v_cont, rwk, rwv, my_lutk, my_lutv, one, ktile, vtile, q16,
                                   my_obuf, lane, G, sacc, pb_hi, pb_lo);
        else if (wv)
            wide_pass<false, true, PAIRS>(ck, cv, ringk, ringv, p.k_cont, p.v_cont, rwk, rwv, my_lutk, my_lutv, one, ktile, vtile, q16,
                                   my_obuf, lane, G, sacc, pb_hi, pb_lo);

        // The item descriptors are derived again rather than kept in registers across the pass.
        cur = item_of(nK, hint);
        nxt = cur;
        if (last_head) nxt = item_of(nK + 1, cur.b);
        tok0 = (cur.blk * nw + warp) * kChunk;
        wk = cur.valid && tok0 < cur.len;

        // streams that ended with this pass hand their ring to the next item's streams
        cp_async_wait<0>();
        __syncwarp();
        // (the V streams of the previous item, if any, ended with this pass: V runs one step behind K)
        if (cur.valid && kK == 0) start_chain(cv, nK, cur, p.v_cont, rwv, ringv, kRowsV);
        if (cur.valid && last_head) start_chain(ck, nK + 1, nxt, p.k_cont, rwk, ringk, kRowsK);
        cp_async_commit();

        // ------------------------------------------ logits of this step's head and the warp's maximum (base 2)
        float lg[4][2], sv_t[4][2], ov_t[4][2];
        if (cur.valid) {
            {   // per-token (sK, oK, sV, oV) from token-per-lane to the accumulator layout, through the K tile
                const float sK = __half2float(__ushort_as_half((unsigned short)(hk & 0xffffu)));
                const float oK = __half2float(__ushort_as_half((unsigned short)(hk >> 16)));
                const float sV = __half2float(__ushort_as_half((unsigned short)(hv & 0xffffu)));
                const float oV = __half2float(__ushort_as_half((unsigned short)(hv >> 16)));
                // the key scale carries the logit scale (sm_scale * log2 e): logits come out in base-2 units
                asm volatile("st.shared.v4.f32 [%0], {%1,%2,%3,%4};\n" ::"r"(ktile + lane * 16), "f"(sK * p.scale_log2), "f"(oK),
                             "f"(sV), "f"(oV) : "memory");
            }
            int row_len = cur.len;   // tokens this thread's row may see (earlier query tokens stop earlier)
            if (p.q_total > 1) row_len -= max(0, row_offset(p, g_row) - (p.resid_lens ? max(p.resid_lens[cur.b], 0) : 0));
            float qmu = 0.f, qs = 0.f;   // both times the logit scale
            if (g_row < G) {
                qs = qsum[(s & 1) * DQ_MAX_GROUP + g_row] * p.scale_log2;
                if (p.has_mean && tok0 < cur.len) qmu = __uint_as_float(lds32(my_qmu + ((s & 1) * DQ_MAX_GROUP + g_row) * 4)) * p.scale_log2;
            }
            __syncwarp();
            float mx = -INFINITY;
            const uint32_t meta = ktile + 2 * qd * 16;
            if (tok0 + kChunk <= row_len) {   // every token of the chunk is visible: no masks
#pragma unroll
                for (int i = 0; i < 4; ++i)
#pragma unroll
                    for (int u = 0; u < 2; ++u) {
                        float4 m4;
                        asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];\n"
                                     : "=f"(m4.x), "=f"(m4.y), "=f"(m4.z), "=f"(m4.w) : "r"(meta + (8 * i + u) * 16));
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
                                     : "=f"(m4.x), "=f"(m4.y), "=f"(m4.z), "=f"(m4.w) : "r"(meta + (8 * i + u) * 16));
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
        __syncthreads();   // output slots of the V step complete; chunk maxima of the K step published

        // ------------------------------------------ finish the V step: sum the warps' slots, write the partial
        if (have_prev) {
            // G x 32 threads add the channel sums four at a time, 2 G more the (l, off) columns (by step parity)
            const int par = (s + 1) & 1;
            const float* slots = reinterpret_cast<const float*>(smem + kOffWarp + kWObuf);
            const int wfl = wstride / 4;   // floats between the slots of neighbouring warps
            for (int e = tid; e < G * 34; e += nthreads) {
                if (e < G * 32) {
                    const int g = e >> 5, c4 = e & 31;
                    const float* src = slots + g * kORow + 4 * c4;
                    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
                    for (int w = 0; w < nwv; ++w) {
                        const float4 v = *reinterpret_cast<const float4*>(src + w * wfl);
                        acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
                    }
                    *reinterpret_cast<float4*>(p.partial + ((size_t)s_prev_row[par] + g) * kPartial + 4 * c4) = acc;
                } else {
                    const int e2 = e - G * 32, g = e2 >> 1, which = e2 & 1;
                    const float* src = slots + g * kORow + kN + 2 * par + which;
                    float acc = 0.f;
                    for (int w = 0; w < nwv; ++w) acc += src[w * wfl];
                    float* dst = p.partial + ((size_t)s_prev_row[par] + g) * kPartial;
                    dst[kN + 1 + which] = acc;
                    if (which == 0) dst[kN] = red_M[par * DQ_MAX_GROUP + g];
                }
            }
        }

        // ------------------------------------------ softmax weights of this step, scaled by the step maximum
        have_prev = cur.valid;
        kV = kK;
        wv = wk;
        nwv = min(nw, (cur.len - cur.blk * nw * kChunk + kChunk - 1) / kChunk);
        if (cur.valid) {
            float m_item = -INFINITY;   // the four threads of a head row share the warps' maxima
            for (int w = qd; w < nw; w += 4) m_item = fmaxf(m_item, red_m[w * DQ_MAX_GROUP + g_row]);
            m_item = fmaxf(m_item, __shfl_xor_sync(kFullMask, m_item, 1));
            m_item = fmaxf(m_item, __shfl_xor_sync(kFullMask, m_item, 2));
            if (warp == 0 && qd == 0) red_M[(s & 1) * DQ_MAX_GROUP + g_row] = m_item;
            const float m_use = (m_item == -INFINITY) ? 0.f : m_item;
            float lsum = 0.f, osum = 0.f;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                float ps[2];
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                    const float pr = ex2_approx(lg[i][u] - m_use);
                    lsum += pr;
                    osum = fmaf(pr, ov_t[i][u], osum);
                    ps[u] = pr * sv_t[i][u];
                }
                const __half2 h2 = __floats2half2_rn(ps[0], ps[1]);   // fp16 hi + lo pair of each weight
                const float2 hf = __half22float2(h2);
                pb_hi[i >> 1][i & 1] = *reinterpret_cast<const uint32_t*>(&h2);
                pb_lo[i >> 1][i & 1] = pack_half2(ps[0] - hf.x, ps[1] - hf.y);
            }
            lsum += __shfl_xor_sync(kFullMask, lsum, 1);
            lsum += __shfl_xor_sync(kFullMask, lsum, 2);
            osum += __shfl_xor_sync(kFullMask, osum, 1);
            osum += __shfl_xor_sync(kFullMask, osum, 2);
            if (qd == 0 && g_row < G) {
                sts32f(my_obuf + (g_row * kORow + kN + 2 * (s & 1)) * 4, lsum);
                sts32f(my_obuf + (g_row * kORow + kN + 2 * (s & 1) + 1) * 4, osum);
            }
        }
        if (tid == 0) s_prev_row[s & 1] = (long long)cur.bg * p.Hq + (long long)(cur.grp * hs + kK) * G;

        // advance the K chain's position
        if (cur.valid) {
            if (last_head) { cur = nxt; ++nK; kK = 0; hint = cur.b; }
            else ++kK;
        }
    }
    cp_async_wait<0>();
    (void)hint;
}

}  // namespace

int dq_attn_wide_pick_warps(const DqDevTable& tk, const DqDevTable& tv, int B, int G, int smem_max) {
    (void)tk; (void)tv;
    for (int nw = kWideWarps; nw >= 4; --nw)
        if (wide_smem_bytes(nw, B, G) <= smem_max) return nw;
    return 0;
}

cudaError_t dq_launch_attention_wide_main(const DqDevTable& tk, const DqDevTable& tv, const AttnParams& p, int nw,
                                          int sm_count, cudaStream_t st) {
    const int smem_bytes = wide_smem_bytes(nw, p.B, p.G);
    auto kernel = tk.pair ? dq_attention_wide_kernel<true> : dq_attention_wide_kernel<false>;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
    if (e != cudaSuccess) return e;
    return dq_launch_pdl(kernel, dim3(sm_count), dim3(nw * 32), (size_t)smem_bytes, st, tk, tv, p);
}
