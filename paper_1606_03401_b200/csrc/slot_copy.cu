// Push / Pop of a memorised state as an explicit copy (Algorithm 2): global -> shared -> global
// through the bulk asynchronous copy engine (untiled TMA), so that a handful of threads keep
// megabytes in flight and the copy runs at the HBM rate.
//
// One CTA per SM; each walks the chunks cta, cta + grid, ... of 32 KB through a ring of four
// shared-memory stages.  A single thread issues everything: the load of a chunk completes on the
// stage's mbarrier, the store of that stage is committed as a bulk group, and a stage is refilled
// once the store that read it has finished reading.  Copies of less than 256 KB take a plain
// vectorised kernel instead (one 16-byte load and store per thread and round): at that size the
// launch, not the bandwidth, is what is paid for.
#include <cuda_runtime.h>

#include <cstdint>

#include "kernels.hpp"
#include "sm100.cuh"

namespace mebptt {
namespace generic {

namespace {

using namespace sm100;

constexpr uint32_t CHUNK = 32 * 1024;
constexpr int STAGES = 4;

__device__ __forceinline__ void bulk_load(void* smem_dst, const void* gsrc, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(smem_u32(smem_dst)), "l"(reinterpret_cast<uint64_t>(gsrc)), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ void bulk_store(void* gdst, const void* smem_src, uint32_t bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
               ::"l"(reinterpret_cast<uint64_t>(gdst)), "r"(smem_u32(smem_src)), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// at most N committed groups may still be reading their shared-memory source
template <int N>
__device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

__global__ void __launch_bounds__(32, 1) slot_copy_bulk(char* dst, const char* src, size_t bytes) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ uint64_t full[STAGES];
  uint8_t* ring = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~uintptr_t(127));
  if (threadIdx.x != 0) return;
  for (int s = 0; s < STAGES; ++s) mbar_init(&full[s], 1);
  mbar_fence_init();

  const size_t nchunks = (bytes + CHUNK - 1) / CHUNK;
  const size_t first = blockIdx.x, stride = gridDim.x;
  // the i-th chunk of this CTA is chunk first + i * stride
  const size_t mine = first < nchunks ? (nchunks - first + stride - 1) / stride : 0;
  auto chunk_off = [&](size_t i) { return (first + i * stride) * (size_t)CHUNK; };
  auto chunk_len = [&](size_t i) {
    const size_t off = chunk_off(i);
    return (uint32_t)(bytes - off < CHUNK ? bytes - off : CHUNK);
  };
  auto load = [&](size_t i) {
    const int s = (int)(i % STAGES);
    mbar_arrive_expect_tx(&full[s], chunk_len(i));
    bulk_load(ring + (size_t)s * CHUNK, src + chunk_off(i), chunk_len(i), &full[s]);
  };
  const size_t ahead = mine < (size_t)(STAGES - 1) ? mine : (size_t)(STAGES - 1);
  for (size_t i = 0; i < ahead; ++i) load(i);
  for (size_t i = 0; i < mine; ++i) {
    const int s = (int)(i % STAGES);
    if (!mbar_wait(&full[s], (uint32_t)(i / STAGES) & 1)) break;   // bounded; a load of mapped memory always lands
    bulk_store(dst + chunk_off(i), ring + (size_t)s * CHUNK, chunk_len(i));
    bulk_commit();
    if (i + STAGES - 1 < mine) {
      // the stage of chunk i - 1 is the one chunk i + STAGES - 1 goes to: its store must have read it
      bulk_wait_read<1>();
      load(i + STAGES - 1);
    }
  }
  bulk_wait_all();
}

__global__ void copy16_small(uint4* dst, const uint4* src, size_t n) {
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x)
    dst[i] = src[i];
}

}  // namespace

void copy_bytes(void* dst, const void* src, size_t bytes, cudaStream_t s) {
  if (bytes < 16) return;
  if (bytes < 256 * 1024) {
    const size_t n = bytes / 16;
    size_t blocks = (n + 255) / 256;
    if (blocks > 148 * 8) blocks = 148 * 8;
    copy16_small<<<(unsigned)blocks, 256, 0, s>>>((uint4*)dst, (const uint4*)src, n);
    return;
  }
  // per call: function attributes belong to the current device
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  cudaFuncSetAttribute(slot_copy_bulk, cudaFuncAttributeMaxDynamicSharedMemorySize, STAGES * CHUNK + 128);
  const size_t nchunks = (bytes + CHUNK - 1) / CHUNK;
  const unsigned grid = (unsigned)(nchunks < (size_t)sms ? nchunks : (size_t)sms);
  slot_copy_bulk<<<grid, 32, STAGES * CHUNK + 128, s>>>((char*)dst, (const char*)src, bytes);
}

}  // namespace generic
}  // namespace mebptt
