// Read-only streaming probe: what this GPU delivers to a kernel that only reads, as a second
// denominator beside the copy bandwidth for the HBM-bound aggregation kernels (which read r*f words
// per word written).  The 64-bit words of a buffer are XOR-ed together, so the loads cannot be
// dropped and the result can be checked exactly.
#include "bz_common.cuh"

namespace bz {

namespace {

constexpr int kProbeBlock = 256;
constexpr int kProbeUnroll = 8;   // 128-bit loads in flight per thread

__global__ void __launch_bounds__(kProbeBlock)
    stream_probe_kernel(const uint4* __restrict__ p, size_t n16, const uint64_t* __restrict__ tail, int n_tail,
                        unsigned long long* __restrict__ checksum) {
    const size_t stride = static_cast<size_t>(gridDim.x) * blockDim.x;
    size_t i = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    uint4 acc = make_uint4(0, 0, 0, 0);
    for (; i + (kProbeUnroll - 1) * stride < n16; i += kProbeUnroll * stride) {
        uint4 x[kProbeUnroll];
#pragma unroll
        for (int u = 0; u < kProbeUnroll; ++u) x[u] = __ldcs(p + i + u * stride);
#pragma unroll
        for (int u = 0; u < kProbeUnroll; ++u) {
            acc.x ^= x[u].x;
            acc.y ^= x[u].y;
            acc.z ^= x[u].z;
            acc.w ^= x[u].w;
        }
    }
    for (; i < n16; i += stride) {
        const uint4 x = __ldcs(p + i);
        acc.x ^= x.x;
        acc.y ^= x.y;
        acc.z ^= x.z;
        acc.w ^= x.w;
    }
    unsigned long long w = (static_cast<unsigned long long>(acc.y ^ acc.w) << 32) | (acc.x ^ acc.z);
    if (blockIdx.x == 0 && threadIdx.x < n_tail) w ^= tail[threadIdx.x];  // a last 64-bit word past the 16-byte units
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) w ^= __shfl_xor_sync(0xffffffffu, w, o);
    __shared__ unsigned long long part[kProbeBlock / 32];
    if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = w;
    __syncthreads();
    if (threadIdx.x == 0) {
        unsigned long long s = 0;
        for (int k = 0; k < kProbeBlock / 32; ++k) s ^= part[k];
        atomicXor(checksum, s);
    }
}

}  // namespace

}  // namespace bz

using namespace bz;

extern "C" int bz_stream_probe(const void* buf, size_t bytes, uint64_t* checksum, void* stream) {
    if (checksum == nullptr || (buf == nullptr && bytes > 0)) return BZ_ERR_INVALID_ARG;
    if (!aligned16(buf) || (bytes % 8) != 0) return BZ_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaMemsetAsync(checksum, 0, sizeof(uint64_t), s);
    if (e != cudaSuccess) return cuda_failed(e);
    if (bytes == 0) return BZ_OK;
    const size_t n16 = bytes / 16;
    const int n_tail = static_cast<int>((bytes % 16) / 8);
    size_t blocks = (n16 + kProbeBlock - 1) / kProbeBlock;
    if (blocks > static_cast<size_t>(kNumSMs) * 8) blocks = static_cast<size_t>(kNumSMs) * 8;
    if (blocks < 1) blocks = 1;
    stream_probe_kernel<<<static_cast<unsigned>(blocks), kProbeBlock, 0, s>>>(
        static_cast<const uint4*>(buf), n16, reinterpret_cast<const uint64_t*>(static_cast<const char*>(buf) + n16 * 16), n_tail,
        reinterpret_cast<unsigned long long*>(checksum));
    note_launch();
    return check_launch();
}
