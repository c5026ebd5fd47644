// Replica parameter executor (paper, "Device-initiated replica transfers"): copies driven by the
// device-resident replica map, with no host read of the plan.
//
//   pull (forward):          replica_buf[r][j]            <- main_params[main(e)][l(e)]
//   gradient return (bwd):   grad_acc[main(e)][r][l(e)]   <- replica_buf[r][j]
//
// for every occupied slot (r, j), e = replica_map[r][j].  Both are one batch of |W|-byte block
// copies whose sources and destinations are known only on the device.  The work is pure HBM
// traffic: |W| bytes read and |W| written per occupied slot.
//
// Every CTA first compacts the occupied slots into the same (source block, destination block)
// list in shared memory, cuts each block into chunks and takes the chunks
// blockIdx.x, blockIdx.x + gridDim.x, ...: an even split without atomics, whatever slots are
// empty.  Two copy engines:
//   bulk  (default) one thread per CTA drives a ring of shared-memory stages with the bulk
//         asynchronous copy unit: cp.async.bulk global->shared completing on an mbarrier, then
//         cp.async.bulk shared->global tracked as a bulk group.  No registers or load/store
//         issue slots are spent on the data.
//   plain 256 threads move 16-byte words with ordinary loads and stores.
// The waits on the mbarriers are bounded: a wait that runs out sets TOPOEP_FLAG_INTERNAL, and the
// thread stops issuing, drains its own stores and returns.
#include "topoep_internal.cuh"

namespace topoep {

namespace {

// Measured on B200 for 32 blocks of 88 MB: 32 KiB x 3 stages 0.955 of the copy peak,
// 16 KiB x 6 0.942, 8 KiB x 12 0.937 (two CTAs per SM each); four CTAs of 16 KiB x 3 0.942.
constexpr int kStageBytes = 32 * 1024;   // one chunk = one ring stage
constexpr int kStages = 3;               // 96 KiB of ring per CTA
constexpr int kBulkCtasPerSm = 2;
constexpr int kBulkThreads = 32;
constexpr int kPlainThreads = 256;
constexpr unsigned kWaitLimit = 1u << 22;   // polls (about 0.1 s) before a wait is given up
constexpr unsigned kSelfTestWaitLimit = 1u << 12;   // the self test's wait, which cannot succeed

struct CopyPair { uint32_t src, dst; };   // block indices, in units of |W| bytes

// Compact the occupied slots of the plan into list[]; every warp of every CTA derives the same
// order (ascending slot index).  Returns the number of occupied slots.  Called by warp 0.
template <int DIR>
__device__ int build_list(const TransferParams& p, CopyPair* list, int lane) {
  const Dims& d = p.d;
  const int slots = d.R * d.N;
  int n = 0;
  for (int base = 0; base < slots; base += 32) {
    const int idx = base + lane;
    int e = -1;
    if (idx < slots) e = p.replica_map[idx];
    if (e >= d.E) {   // not an expert id: leave the slot alone and report it
      atomicOr(p.ws.status, TOPOEP_FLAG_BAD_ID);
      e = -1;
    }
    const bool occ = e >= 0;
    const unsigned m = __ballot_sync(0xffffffffu, occ);
    if (occ) {
      const int r = idx / d.N;
      const uint32_t main_block = (uint32_t)(p.ws.main_rank[e] * d.e_loc + p.ws.main_local[e]);
      CopyPair cp;
      if (DIR == 0) {   // pull: main block -> slot
        cp.src = main_block;
        cp.dst = (uint32_t)idx;
      } else {          // gradient return: slot -> region [main rank][source rank][local]
        cp.src = (uint32_t)idx;
        cp.dst = (uint32_t)((p.ws.main_rank[e] * d.R + r) * d.e_loc + p.ws.main_local[e]);
      }
      list[n + __popc(m & lanemask_lt())] = cp;
    }
    n += __popc(m);
  }
  return n;
}

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}

__device__ __forceinline__ void bulk_load(uint32_t dst_smem, const void* src, uint32_t bytes,
                                          uint32_t bar) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
               : "memory");
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::
          "r"(dst_smem), "l"(src), "r"(bytes), "r"(bar)
      : "memory");
}

__device__ __forceinline__ void bulk_store(void* dst, uint32_t src_smem, uint32_t bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst),
               "r"(src_smem), "r"(bytes)
               : "memory");
  asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}

// Bounded wait for the phase with the given parity; false if it ran out after `limit` polls.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, unsigned limit) {
  for (unsigned i = 0; i < limit; ++i) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(bar), "r"(parity)
        : "memory");
    if (done) return true;
  }
  return false;
}

template <int DIR>
__global__ void __launch_bounds__(kBulkThreads) transfer_bulk_kernel(const TransferParams p) {
  extern __shared__ __align__(128) unsigned char smem[];
  __shared__ __align__(8) unsigned long long bars[kStages];
  unsigned char* ring = smem;                                             // kStages * kStageBytes
  CopyPair* list = reinterpret_cast<CopyPair*>(smem + kStages * kStageBytes);
  const int lane = threadIdx.x;
  const int n_occ = build_list<DIR>(p, list, lane);
  if (lane == 0) {
    for (int s = 0; s < kStages; ++s)
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&bars[s])) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncwarp();
  if (lane != 0 || n_occ == 0 || p.param_bytes == 0) return;

  const unsigned long long W = p.param_bytes;
  const unsigned long long chunks = (W + kStageBytes - 1) / kStageBytes;   // per block
  const unsigned long long items = chunks * (unsigned long long)n_occ;
  const unsigned long long first = blockIdx.x, step = gridDim.x;
  if (first >= items) return;
  const unsigned long long mine = (items - first + step - 1) / step;
  const unsigned char* src_base = static_cast<const unsigned char*>(p.src);
  unsigned char* dst_base = static_cast<unsigned char*>(p.dst);

  // item n of this CTA -> (addresses, bytes); chunk-major order so that neighbouring CTAs stream
  // through neighbouring chunks of the same block
  auto locate = [&](unsigned long long n, const unsigned char** s, unsigned char** d,
                    uint32_t* bytes) {
    const unsigned long long it = first + n * step;
    const unsigned long long blk = it / chunks, c = it - blk * chunks;
    const CopyPair cp = list[blk];
    const unsigned long long off = c * kStageBytes;
    *bytes = (uint32_t)min((unsigned long long)kStageBytes, W - off);
    *s = src_base + (unsigned long long)cp.src * W + off;
    *d = dst_base + (unsigned long long)cp.dst * W + off;
  };

  // Self test of the give-up path (host knob, tests only): CTA 0 announces the bytes of its first
  // chunk on the stage's barrier but never issues the copy, so nothing is in flight for that
  // stage, its wait runs out after a short limit, and the CTA must flag, drain and return.
  const bool selftest = p.selftest != 0 && blockIdx.x == 0;
  const unsigned limit = selftest ? kSelfTestWaitLimit : kWaitLimit;
  const unsigned long long lead = min((unsigned long long)(kStages - 1), mine);
  unsigned long long issued = 0;   // items whose load has been handed to the copy unit
  for (unsigned long long n = 0; n < lead; ++n) {
    const unsigned char* s; unsigned char* d; uint32_t bytes;
    locate(n, &s, &d, &bytes);
    if (selftest && n == 0) {
      asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(&bars[0])),
                   "r"(bytes)
                   : "memory");
    } else {
      bulk_load(smem_u32(ring + (n % kStages) * kStageBytes), s, bytes, smem_u32(&bars[n % kStages]));
    }
    issued = n + 1;
  }
  for (unsigned long long n = 0; n < mine; ++n) {
    const int st = (int)(n % kStages);
    if (!mbar_wait(smem_u32(&bars[st]), (uint32_t)((n / kStages) & 1), limit)) {
      // Gave up on item n: report it, issue nothing more, and let the loads already handed to the
      // copy unit land (bounded waits again) so that none is still writing this CTA's shared
      // memory when it exits; the stores are drained below.
      atomicOr(p.ws.status, TOPOEP_FLAG_INTERNAL);
      for (unsigned long long m = n + 1; m < issued; ++m)
        mbar_wait(smem_u32(&bars[m % kStages]), (uint32_t)((m / kStages) & 1), kWaitLimit);
      break;
    }
    const unsigned char* s; unsigned char* d; uint32_t bytes;
    locate(n, &s, &d, &bytes);
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    bulk_store(d, smem_u32(ring + st * kStageBytes), bytes);
    // the stage of item n-1 is free once its store has read it (all groups but the newest);
    // refill it with item n-1+kStages
    const unsigned long long nx = n + kStages - 1;
    if (nx < mine) {
      asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
      locate(nx, &s, &d, &bytes);
      bulk_load(smem_u32(ring + (nx % kStages) * kStageBytes), s, bytes,
                smem_u32(&bars[nx % kStages]));
      issued = nx + 1;
    }
  }
  asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
}

template <int DIR>
__global__ void __launch_bounds__(kPlainThreads) transfer_plain_kernel(const TransferParams p) {
  extern __shared__ __align__(128) unsigned char smem[];
  __shared__ int n_shared;
  CopyPair* list = reinterpret_cast<CopyPair*>(smem);
  if (threadIdx.x < 32) {
    const int n = build_list<DIR>(p, list, threadIdx.x);
    if (threadIdx.x == 0) n_shared = n;
  }
  __syncthreads();
  const int n_occ = n_shared;
  const unsigned long long W = p.param_bytes;
  if (n_occ == 0 || W == 0) return;
  const unsigned long long chunks = (W + kStageBytes - 1) / kStageBytes;
  const unsigned long long items = chunks * (unsigned long long)n_occ;
  const unsigned char* src_base = static_cast<const unsigned char*>(p.src);
  unsigned char* dst_base = static_cast<unsigned char*>(p.dst);
  constexpr int kVec = kStageBytes / 16 / kPlainThreads;   // 16-byte words per thread and chunk
  for (unsigned long long it = blockIdx.x; it < items; it += gridDim.x) {
    const unsigned long long blk = it / chunks, c = it - blk * chunks;
    const CopyPair cp = list[blk];
    const unsigned long long off = c * kStageBytes;
    const int words = (int)(min((unsigned long long)kStageBytes, W - off) / 16);
    const int4* s = reinterpret_cast<const int4*>(src_base + (unsigned long long)cp.src * W + off);
    int4* d = reinterpret_cast<int4*>(dst_base + (unsigned long long)cp.dst * W + off);
    int4 v[kVec];
#pragma unroll
    for (int i = 0; i < kVec; ++i) {
      const int w = threadIdx.x + i * kPlainThreads;
      if (w < words) v[i] = __ldcs(s + w);
    }
#pragma unroll
    for (int i = 0; i < kVec; ++i) {
      const int w = threadIdx.x + i * kPlainThreads;
      if (w < words) __stcs(d + w, v[i]);
    }
  }
}

size_t list_bytes(const Dims& d) { return ((size_t)d.R * d.N * sizeof(CopyPair) + 127) / 128 * 128; }

}  // namespace

size_t transfer_smem_bytes(const Dims& d, int mode) {
  return list_bytes(d) + (mode == 0 ? (size_t)kStages * kStageBytes : 0);
}

cudaError_t configure_transfer(const Dims& d) {
  cudaError_t e;
  const int bulk = (int)transfer_smem_bytes(d, 0), plain = (int)transfer_smem_bytes(d, 1);
  if ((e = cudaFuncSetAttribute(transfer_bulk_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, bulk)) != cudaSuccess) return e;
  if ((e = cudaFuncSetAttribute(transfer_bulk_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, bulk)) != cudaSuccess) return e;
  if ((e = cudaFuncSetAttribute(transfer_plain_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, plain)) != cudaSuccess) return e;
  return cudaFuncSetAttribute(transfer_plain_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, plain);
}

cudaError_t launch_transfer(const TransferParams& p, int direction, int mode, int sms,
                            cudaStream_t stream) {
  const size_t smem = transfer_smem_bytes(p.d, mode);
  if (mode == 0) {
    const dim3 grid(kBulkCtasPerSm * sms), block(kBulkThreads);
    if (direction == 0) transfer_bulk_kernel<0><<<grid, block, smem, stream>>>(p);
    else transfer_bulk_kernel<1><<<grid, block, smem, stream>>>(p);
  } else {
    const dim3 grid(8 * sms), block(kPlainThreads);
    if (direction == 0) transfer_plain_kernel<0><<<grid, block, smem, stream>>>(p);
    else transfer_plain_kernel<1><<<grid, block, smem, stream>>>(p);
  }
  return cudaGetLastError();
}

}  // namespace topoep
