// Chained launches (programmatic dependent launch, sm_90 and later).
//
// A step is a string of a dozen kernels on one stream, several of them a few microseconds long, so the gap between
// the end of one kernel and the first instruction of the next is a measurable part of it.  A kernel launched with the
// programmatic-serialization attribute may become resident before its predecessor in the stream has completed:
//   - by default as soon as all of the predecessor's blocks have exited (its completion and memory flush still pending);
//   - earlier, if every block of the predecessor calls chain_release(): then the successor's blocks take the slots
//     that the predecessor's blocks free one by one;
//   - the successor does what needs no global memory (shared-memory clears, hashes from the parameters), then calls
//     chain_acquire(), which returns once every kernel before it in the stream has completed and its writes are
//     visible.
// Rules kept by every kernel that is launched this way:
//   - no global memory is read or written before chain_acquire();
//   - chain_acquire() is reached by every block, before any early return, so that the completion of a kernel always
//     implies the completion of all kernels before it (the property its own successor relies on);
//   - chain_release() is called only by the persistent kernels whose whole grid is resident from their start (the
//     shared-memory sketch kernel, the windowed key pass, the emit pass).  Measured: with an early release in the
//     short multi-wave kernels too (table clears, sums, the one-block kernels), blocks of later kernels took slots
//     that pending blocks of earlier ones needed, and a step with several sketch launches ran 17 % slower.
// Both calls do nothing in a kernel launched without the attribute, and a kernel launched without the attribute after
// one that released is serialised as usual, so chained and plain launches mix freely.
#pragma once
#include <cuda_runtime.h>
#include <cstdint>

namespace sk {

// which launches of a step are chained (bits of Params::chain)
constexpr uint32_t kChainZero = 1u, kChainSketch = 2u, kChainSum = 4u, kChainKeys = 8u, kChainPick = 16u, kChainEmit = 32u,
                   kChainRefine = 64u, kChainApply = 128u, kChainExact = 256u, kChainAll = 511u;

__device__ __forceinline__ void chain_release() { asm volatile("griddepcontrol.launch_dependents;"); }
__device__ __forceinline__ void chain_acquire() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Launches kfn(args...) on st; chain = true adds the programmatic-serialization attribute.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel(bool chain, void (*kfn)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                 Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = chain ? 1u : 0u;
    return cudaLaunchKernelEx(&cfg, kfn, static_cast<KArgs>(args)...);
}

}  // namespace sk
