// Gather micro-benchmark: the row gather of the decode kernel, alone, done three ways.
//
// The decode kernel reads selected cache rows (256 bytes each at D = 128) with per-lane 256-bit loads.  The
// alternative for rows that are contiguous within a span is a bulk asynchronous copy (cp.async.bulk, the
// untiled TMA form) from global to shared memory, completion signalled on an mbarrier.  This file times the
// data movement alone, on the same lists of rows:
//   mode 0  plain loads: 8 lanes x 32 bytes per row, 8 loads in flight per lane (what the kernel does)
//   mode 1  bulk copies into a shared-memory ring that the block's threads then read: one copy per run of
//           `run_rows` consecutive rows (1 = a copy per 256-byte row ... 32 = one 8 KB copy per stage)
// The unit of work is a "stage": 32 rows = 8 KB.  Every byte that arrives is folded into a checksum, so the
// three modes can be checked against one another.  Bulk copies never use multicast and only ever read this
// GPU's memory.  Every wait on an mbarrier is bounded: on expiry the block raises an error flag, stops
// issuing, drains what it has in flight (bounded again) and returns.
#include <cuda_runtime.h>
#include <stdint.h>

namespace {

constexpr int kRowBytes = 256;
constexpr int kStageRows = 32;
constexpr int kStageBytes = kRowBytes * kStageRows;   // 8 KB
constexpr int kThreads = 128;
constexpr uint32_t kSpinLimit = 1u << 20;             // try_wait attempts before a wait gives up

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(bar)) : "memory");
}
// Bounded wait for the phase with the given parity to complete.  false: gave up.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) {
  for (uint32_t spin = 0; spin < kSpinLimit; ++spin) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(smem_addr(bar)), "r"(parity)
        : "memory");
    if (done) return true;
  }
  return false;
}
// Untiled bulk copy global -> this block's shared memory; both addresses 16-byte aligned, bytes a multiple of 16.
__device__ __forceinline__ void bulk_copy(void* dst_smem, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(smem_addr(dst_smem)), "l"(src), "r"(bytes), "r"(smem_addr(bar))
               : "memory");
}

__device__ __forceinline__ uint32_t fold(uint4 v) { return v.x ^ v.y ^ v.z ^ v.w; }

// mode 0: every warp takes stages warp, warp + n_warps, ...; a stage is 8 loads of 32 bytes per lane.
__global__ void __launch_bounds__(kThreads) gather_loads_kernel(const char* __restrict__ buf, const int32_t* __restrict__ rows,
                                                                int n_stages, uint32_t* checksum) {
  const int lane = threadIdx.x & 31, col = lane & 7, sub = lane >> 3;
  const int warp = (blockIdx.x * kThreads + threadIdx.x) >> 5, n_warps = (gridDim.x * kThreads) >> 5;
  uint32_t sum = 0;
  for (int s = warp; s < n_stages; s += n_warps) {
    const int32_t my_row = rows[s * kStageRows + lane];
    uint32_t w[8][8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int32_t r = __shfl_sync(0xffffffffu, my_row, u * 4 + sub);
      const char* p = buf + (size_t)r * kRowBytes + col * 32;
      asm volatile("ld.global.nc.L1::no_allocate.L2::evict_first.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                   : "=r"(w[u][0]), "=r"(w[u][1]), "=r"(w[u][2]), "=r"(w[u][3]), "=r"(w[u][4]), "=r"(w[u][5]),
                     "=r"(w[u][6]), "=r"(w[u][7])
                   : "l"(p));
    }
#pragma unroll
    for (int u = 0; u < 8; ++u)
#pragma unroll
      for (int i = 0; i < 8; ++i) sum ^= w[u][i];
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) sum ^= __shfl_xor_sync(0xffffffffu, sum, o);
  if (lane == 0 && sum) atomicXor(checksum, sum);
}

// mode 1: a ring of `stages` 8 KB buffers per block.  Thread 0 is the producer (arms the stage's "full"
// barrier with the byte count and issues the copies); all 128 threads are consumers (read the stage, fold it,
// arrive on its "empty" barrier).  The producer runs up to `stages` stages ahead of the consumers.
__global__ void __launch_bounds__(kThreads) gather_bulk_kernel(const char* __restrict__ buf, const int32_t* __restrict__ rows,
                                                               int n_stages, int stages, int run_rows,
                                                               uint32_t* checksum, uint32_t* error) {
  extern __shared__ __align__(128) unsigned char smem[];
  uint64_t* full = reinterpret_cast<uint64_t*>(smem);
  uint64_t* empty = full + stages;
  unsigned char* ring = smem + 1024;                    // barriers: 2 * stages * 8 bytes <= 1024
  __shared__ int s_abort;
  const int tid = threadIdx.x;
  if (tid == 0) {
    for (int i = 0; i < stages; ++i) {
      mbar_init(&full[i], 1);
      mbar_init(&empty[i], kThreads);
    }
    s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  const int first = blockIdx.x, stride = gridDim.x;
  const int mine = first < n_stages ? (n_stages - first + stride - 1) / stride : 0;   // stages of this block
  uint32_t sum = 0;
  int issued = 0;
  auto produce = [&](int k) {                           // thread 0 only: stage k of this block into slot k % stages
    const int slot = k % stages;
    const int32_t* list = rows + (size_t)(first + (size_t)k * stride) * kStageRows;
    unsigned char* dst = ring + (size_t)slot * kStageBytes;
    mbar_expect_tx(&full[slot], kStageBytes);
    for (int r = 0; r < kStageRows; r += run_rows)      // rows r .. r + run_rows - 1 of the list are consecutive
      bulk_copy(dst + r * kRowBytes, buf + (size_t)list[r] * kRowBytes, (uint32_t)(run_rows * kRowBytes), &full[slot]);
  };
  if (tid == 0)
    for (; issued < mine && issued < stages; ++issued) produce(issued);
  bool ok = true;
  int k = 0;
  for (; k < mine && ok; ++k) {
    const int slot = k % stages;
    const uint32_t phase = (uint32_t)(k / stages) & 1u;
    ok = mbar_wait(&full[slot], phase);
    if (!ok) break;
    const uint4* src = reinterpret_cast<const uint4*>(ring + (size_t)slot * kStageBytes);
#pragma unroll
    for (int i = 0; i < kStageBytes / 16 / kThreads; ++i) sum ^= fold(src[tid + i * kThreads]);
    mbar_arrive(&empty[slot]);
    if (tid == 0 && issued < mine) {                    // refill the slot once everybody has left it
      if (mbar_wait(&empty[slot], phase)) produce(issued++);
      else ok = false;
    }
  }
  if (!ok) {
    atomicExch(&s_abort, 1);
    atomicOr(error, 1u);
  }
  __syncthreads();
  if (s_abort && tid == 0) {
    // something gave up: nothing more is issued; give the copies already in flight a bounded time to land
    // before the block (and its shared memory) goes away
    for (int j = k; j < issued; ++j)
      if (!mbar_wait(&full[j % stages], (uint32_t)(j / stages) & 1u)) break;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) sum ^= __shfl_xor_sync(0xffffffffu, sum, o);
  if ((tid & 31) == 0 && sum) atomicXor(checksum, sum);
}

}  // namespace

extern "C" {

// Runs one launch of the gather in the given mode on `stream`.
//   buf        dev, the cache stand-in: rows of 256 bytes, 256-byte aligned
//   rows       dev int32 [n_stages * 32] row numbers (all inside buf; the caller guarantees it); in mode 1
//              every aligned group of run_rows entries must name consecutive rows
//   grid       thread blocks (128 threads each); stages: ring depth of mode 1 (1..27);
//              run_rows in {1, 2, 4, 8, 16, 32}
//   checksum   dev uint32 [1], XOR-ed with every 32-bit word gathered;  error  dev uint32 [1], set to 1 if a
//              bounded wait expired
// Returns 0, or a cudaError_t / -1 for bad arguments; nothing is launched then.
int ssa_probe_gather(int mode, const void* buf, const int32_t* rows, int n_stages, int grid, int stages,
                     int run_rows, uint32_t* checksum, uint32_t* error, void* stream) {
  if (!buf || !rows || !checksum || !error || n_stages <= 0 || grid <= 0) return -1;
  if (reinterpret_cast<uintptr_t>(buf) % 256 != 0) return -1;
  cudaStream_t st = (cudaStream_t)stream;
  if (mode == 0) {
    gather_loads_kernel<<<grid, kThreads, 0, st>>>(static_cast<const char*>(buf), rows, n_stages, checksum);
    return (int)cudaGetLastError();
  }
  if (mode != 1 || stages < 1 || stages > 27) return -1;
  if (run_rows < 1 || run_rows > kStageRows || (run_rows & (run_rows - 1)) != 0) return -1;
  const size_t smem = 1024 + (size_t)stages * kStageBytes;
  if (smem > 227 * 1024) return -1;
  cudaError_t err = cudaFuncSetAttribute(gather_bulk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (err != cudaSuccess) return (int)err;
  gather_bulk_kernel<<<grid, kThreads, smem, st>>>(static_cast<const char*>(buf), rows, n_stages, stages,
                                                   run_rows, checksum, error);
  return (int)cudaGetLastError();
}

}  // extern "C"
