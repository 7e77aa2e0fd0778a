// Read-only streaming probe: what this GPU delivers to a kernel that only reads, as a second
// denominator beside the copy bandwidth for the HBM-bound aggregation kernels (which read r*f words
// per word written).  The 64-bit words of a buffer are XOR-ed together, so the loads cannot be
// dropped and the result can be checked exactly.
#include "tma_pipeline.cuh"

namespace bz {

__device__ unsigned int g_probe_timeouts = 0;

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

// The same checksum with the bytes brought in by the bulk-copy engine: one producer thread per CTA keeps a
// ring of kRingStages chunks of kRingChunk bytes in flight (cp.async.bulk, completion on mbarriers), four warps
// XOR each chunk out of shared memory.  This is how the staged aggregation kernels read, without their
// arithmetic: the bandwidth it reaches is their ceiling.  Every wait is bounded.
constexpr int kRingChunk = 32768;
constexpr int kRingStages = 4;
constexpr int kRingConsumers = 128;

__device__ __forceinline__ void bulk_load(void* smem_dst, const void* src, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(smem_u32(smem_dst)),
                 "l"(src), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}

__global__ void __launch_bounds__(kRingConsumers + 32)
    stream_probe_ring_kernel(const unsigned char* __restrict__ p, size_t n_chunks, unsigned long long* __restrict__ checksum) {
    extern __shared__ __align__(128) unsigned char ring[];
    uint64_t* full = reinterpret_cast<uint64_t*>(ring + kRingStages * kRingChunk);
    uint64_t* empty = full + kRingStages;
    const int tid = threadIdx.x;
    if (tid == 0) {
        for (int s = 0; s < kRingStages; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], kRingConsumers / 32);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    const size_t mine = blockIdx.x < n_chunks ? (n_chunks - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;
    if (tid >= kRingConsumers) {
        if (tid == kRingConsumers) {
            size_t issued = 0;
            bool alive = true;
            for (; issued < mine && alive; ++issued) {
                const int s = static_cast<int>(issued % kRingStages);
                const uint32_t round = static_cast<uint32_t>(issued / kRingStages);
                if (round > 0 && !mbar_wait(&empty[s], (round - 1) & 1)) {
                    alive = false;
                    break;
                }
                mbar_expect_tx(&full[s], kRingChunk);
                bulk_load(ring + static_cast<size_t>(s) * kRingChunk, p + (blockIdx.x + issued * gridDim.x) * kRingChunk, kRingChunk, &full[s]);
            }
            if (!alive) {
                atomicAdd(&g_probe_timeouts, 1u);
                for (size_t it = issued > kRingStages ? issued - kRingStages : 0; it < issued; ++it)
                    mbar_wait(&full[it % kRingStages], static_cast<uint32_t>(it / kRingStages) & 1);
            }
        }
    } else {
        uint4 acc = make_uint4(0, 0, 0, 0);
        bool alive = true;
        for (size_t it = 0; it < mine && alive; ++it) {
            const int s = static_cast<int>(it % kRingStages);
            if (!mbar_wait(&full[s], static_cast<uint32_t>(it / kRingStages) & 1)) {
                alive = false;
                break;
            }
            const uint4* src = reinterpret_cast<const uint4*>(ring + static_cast<size_t>(s) * kRingChunk);
#pragma unroll
            for (int k = 0; k < kRingChunk / 16 / kRingConsumers; ++k) {
                const uint4 x = src[k * kRingConsumers + tid];
                acc.x ^= x.x;
                acc.y ^= x.y;
                acc.z ^= x.z;
                acc.w ^= x.w;
            }
            __syncwarp();
            if ((tid & 31) == 0) mbar_arrive(&empty[s]);
        }
        if (!alive && (tid & 31) == 0) atomicAdd(&g_probe_timeouts, 1u);
        unsigned long long w = (static_cast<unsigned long long>(acc.y ^ acc.w) << 32) | (acc.x ^ acc.z);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) w ^= __shfl_xor_sync(0xffffffffu, w, o);
        if ((tid & 31) == 0) atomicXor(checksum, w);
    }
}

}  // namespace

int probe_timeouts(unsigned int* count) {
    const cudaError_t e = cudaMemcpyFromSymbol(count, g_probe_timeouts, sizeof(unsigned int));
    return e == cudaSuccess ? BZ_OK : cuda_failed(e);
}

}  // namespace bz

using namespace bz;

extern "C" int bz_stream_probe(const void* buf, size_t bytes, int staged, uint64_t* checksum, void* stream) {
    if (checksum == nullptr || (buf == nullptr && bytes > 0)) return BZ_ERR_INVALID_ARG;
    if (!aligned16(buf) || (bytes % 8) != 0) return BZ_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaMemsetAsync(checksum, 0, sizeof(uint64_t), s);
    if (e != cudaSuccess) return cuda_failed(e);
    if (bytes == 0) return BZ_OK;
    const unsigned char* p = static_cast<const unsigned char*>(buf);
    if (staged) {
        // whole chunks through the ring; what is left (less than one chunk) through the plain kernel below
        const size_t n_chunks = bytes / kRingChunk;
        if (n_chunks > 0) {
            constexpr int smem = kRingStages * kRingChunk + 2 * kRingStages * 8;
            e = cudaFuncSetAttribute(stream_probe_ring_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
            if (e != cudaSuccess) return cuda_failed(e);
            const unsigned grid = static_cast<unsigned>(n_chunks < static_cast<size_t>(kNumSMs) ? n_chunks : kNumSMs);
            stream_probe_ring_kernel<<<grid, kRingConsumers + 32, smem, s>>>(p, n_chunks, reinterpret_cast<unsigned long long*>(checksum));
            note_launch();
            const int st = check_launch();
            if (st != BZ_OK) return st;
        }
        p += n_chunks * kRingChunk;
        bytes -= n_chunks * kRingChunk;
        if (bytes == 0) return BZ_OK;
    }
    const size_t n16 = bytes / 16;
    const int n_tail = static_cast<int>((bytes % 16) / 8);
    size_t blocks = (n16 + kProbeBlock - 1) / kProbeBlock;
    if (blocks > static_cast<size_t>(kNumSMs) * 8) blocks = static_cast<size_t>(kNumSMs) * 8;
    if (blocks < 1) blocks = 1;
    stream_probe_kernel<<<static_cast<unsigned>(blocks), kProbeBlock, 0, s>>>(
        reinterpret_cast<const uint4*>(p), n16, reinterpret_cast<const uint64_t*>(p + n16 * 16), n_tail,
        reinterpret_cast<unsigned long long*>(checksum));
    note_launch();
    return check_launch();
}
