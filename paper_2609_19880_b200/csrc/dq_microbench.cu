// Measurement aid: the bare rANS symbol step of the fused attention kernel (Algorithm 2), without
// tiles, tensor-core contractions, softmax or global traffic.  Every lane walks byte streams that
// sit in shared memory through the same decode step the product kernel uses (table address and
// field extraction by dp4a, multiply-add, compare, byte-permute renormalisation) with one or two
// independent chains per lane.  The figure it gives -- clocks per symbol per SM sub-partition --
// is the floor the fused kernel's pass over the channels can be compared with.  The streams are
// arbitrary bytes: a decoder never leaves its state interval whatever it reads, so the instruction
// stream is the product's; the symbols mean nothing.
#include "dq_attention_common.cuh"

using namespace dqdev;
using namespace dqattn;

namespace {

constexpr int kMbRec = 42;   // bytes between the stream starts of neighbouring lanes (the 2.26-bit key record)

__device__ __forceinline__ void mb_decode16(uint32_t& x, uint32_t& ptr, uint32_t lut, uint32_t one, uint32_t (&packed)[8]) {
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
            asm("{.reg .pred p; setp.lt.u32 p, %0, 0x800000; @p prmt.b32 %0, %0, %2, %1; "
                "@p mad.lo.u32 %1, %3, %3, %1;}"
                : "+r"(x), "+r"(sel) : "r"(win), "r"(one));
        }
        ptr += sel - 0x2104u;
        packed[2 * q4] = __byte_perm(e[0], e[1], 0x6521u);
        packed[2 * q4 + 1] = __byte_perm(e[2], e[3], 0x6521u);
    }
}

template <int CHAINS>
__global__ void __launch_bounds__(1024, 1)
dq_mb_decode_loop_kernel(const __grid_constant__ DqDevTable T, const uint8_t* __restrict__ bytes, uint32_t nbytes,
                         int reps, uint32_t* __restrict__ out) {
    extern __shared__ __align__(128) uint8_t smem[];
    uint32_t* lut = reinterpret_cast<uint32_t*>(smem);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nw = blockDim.x >> 5;
    for (int i = tid; i < 256 * 32; i += blockDim.x) lut[i] = T.lut[i >> 5];
    uint8_t* st = smem + 32768;
    const int per_warp = 32 * kMbRec * CHAINS + 160;   // a stream advances by at most 128 + 8 bytes
    for (int i = tid; i < nw * per_warp; i += blockDim.x)
        st[i] = bytes[((size_t)blockIdx.x * nw * per_warp + i) % nbytes];
    __syncthreads();
    const uint32_t sb = smem_addr(smem);
    const uint32_t my_lut = sb + lane * 4;
    const uint32_t one = (sb >> 31) | 1u;
    uint32_t acc = 0;
    for (int r = 0; r < reps; ++r) {
        uint32_t x[CHAINS], ptr[CHAINS];
#pragma unroll
        for (int s = 0; s < CHAINS; ++s) {
            const uint32_t rb = sb + 32768 + warp * per_warp + (s * 32 + lane) * kMbRec;
            x[s] = (lds32_unaligned(rb + 4) | 0x800000u) & 0x7fffffffu;   // any state of the interval [2^23, 2^31)
            ptr[s] = rb + 8;
        }
#pragma unroll 1
        for (int cg = 0; cg < 8; ++cg) {
#pragma unroll
            for (int s = 0; s < CHAINS; ++s) {
                uint32_t pk[8];
                mb_decode16(x[s], ptr[s], my_lut, one, pk);
#pragma unroll
                for (int i = 0; i < 8; ++i) acc ^= pk[i];
            }
        }
#pragma unroll
        for (int s = 0; s < CHAINS; ++s) acc += x[s];
    }
    out[(size_t)blockIdx.x * blockDim.x + tid] = acc;
}

}  // namespace

// Launches the loop on `ctas` CTAs of `threads` threads, `reps` passes of 128 symbols per chain.
cudaError_t dq_launch_microbench_decode_loop(const DqDevTable& t, const uint8_t* bytes, size_t nbytes, int ctas, int threads,
                                             int chains, int reps, uint32_t* out, cudaStream_t st) {
    const size_t smem = 32768 + (size_t)(threads / 32) * (32 * kMbRec * chains + 160) + 256;
    cudaError_t e;
    if (chains == 1) {
        e = cudaFuncSetAttribute(dq_mb_decode_loop_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        dq_mb_decode_loop_kernel<1><<<ctas, threads, smem, st>>>(t, bytes, (uint32_t)nbytes, reps, out);
    } else {
        e = cudaFuncSetAttribute(dq_mb_decode_loop_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        dq_mb_decode_loop_kernel<2><<<ctas, threads, smem, st>>>(t, bytes, (uint32_t)nbytes, reps, out);
    }
    return cudaGetLastError();
}
