// Sensitive parameter mask (Definition 3): indices of the k largest squared-gradient scores,
// ties to the lowest index, output ascending.
//
// Exact selection without sorting: (1) map each fp32 score to a uint32 key whose unsigned order
// is the score order, (2) four 8-bit radix-select passes find the key T of the k-th largest score
// and how many keys equal to T are still needed, (3) an ordered two-level compaction writes, in
// index order, every i with key > T and the first `need` indices with key == T.
// Everything stays on the device; the host only reads a NaN flag at the end.
#include <mutex>

#include "common.cuh"

namespace szo {

constexpr int kSelBlock = 512;
constexpr int kSelItems = 16;                    // scores per thread in the compaction kernels
constexpr int kSelTile = kSelBlock * kSelItems;  // 8192 scores per block

struct SelectState {
  unsigned long long hist[256];
  unsigned long long remaining;   // how many of the keys matching `prefix` are still wanted
  unsigned long long need_equal;  // number of keys == T to take
  uint32_t prefix;                // high bits of the threshold key fixed so far
  uint32_t threshold;             // final key T
  int32_t nan_flag;
  int32_t pad;
};

__device__ __forceinline__ uint32_t score_key(float s, int32_t* nan_flag) {
  if (s != s) {
    *nan_flag = 1;
    return 0u;
  }
  const uint32_t b = __float_as_uint(s + 0.0f);   // -0 -> +0
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

__global__ void select_init_kernel(SelectState* st, unsigned long long k) {
  if (threadIdx.x < 256) st->hist[threadIdx.x] = 0ull;
  if (threadIdx.x == 0) {
    st->remaining = k;
    st->prefix = 0u;
    st->threshold = 0u;
    st->need_equal = 0ull;
    st->nan_flag = 0;
  }
}

// Histogram of byte `shift/8` over the keys whose higher bytes equal the prefix.
__global__ void __launch_bounds__(kSelBlock)
select_hist_kernel(const float* __restrict__ scores, int64_t n, int shift, SelectState* st) {
  __shared__ unsigned int h[256];
  __shared__ int32_t nan_local;
  if (threadIdx.x < 256) h[threadIdx.x] = 0u;
  if (threadIdx.x == 0) nan_local = 0;
  __syncthreads();
  const uint32_t prefix = st->prefix;
  const uint32_t himask = (shift == 24) ? 0u : (0xFFFFFFFFu << (shift + 8));
  const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
  for (int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < n; i += stride) {
    const uint32_t key = score_key(scores[i], &nan_local);
    if ((key & himask) == prefix) atomicAdd(&h[(key >> shift) & 0xFFu], 1u);
  }
  __syncthreads();
  if (threadIdx.x < 256 && h[threadIdx.x]) atomicAdd(&st->hist[threadIdx.x], (unsigned long long)h[threadIdx.x]);
  if (threadIdx.x == 0 && nan_local) st->nan_flag = 1;
}

// Walk the bins from the largest byte down until the wanted rank falls inside one.
__global__ void select_pick_kernel(SelectState* st, int shift) {
  if (threadIdx.x != 0) return;
  unsigned long long rem = st->remaining;
  int b = 255;
  for (; b > 0; --b) {
    const unsigned long long c = st->hist[b];
    if (c >= rem) break;
    rem -= c;
  }
  st->prefix |= static_cast<uint32_t>(b) << shift;
  st->remaining = rem;
  for (int i = 0; i < 256; ++i) st->hist[i] = 0ull;
  if (shift == 0) {
    st->threshold = st->prefix;
    st->need_equal = rem;
  }
}

// Pass A: per-block counts of (key > T) and (key == T).  Block b covers scores
// [b*kSelTile, (b+1)*kSelTile).
__global__ void __launch_bounds__(kSelBlock)
select_count_kernel(const float* __restrict__ scores, int64_t n, const SelectState* st,
                    uint32_t* __restrict__ blk_gt, uint32_t* __restrict__ blk_eq) {
  __shared__ uint32_t s_gt, s_eq;
  if (threadIdx.x == 0) s_gt = s_eq = 0u;
  __syncthreads();
  const uint32_t T = st->threshold;
  const int64_t base = static_cast<int64_t>(blockIdx.x) * kSelTile;
  uint32_t gt = 0, eq = 0;
  int32_t dummy = 0;
  for (int t = 0; t < kSelItems; ++t) {
    const int64_t i = base + static_cast<int64_t>(t) * kSelBlock + threadIdx.x;
    if (i < n) {
      const uint32_t key = score_key(scores[i], &dummy);
      gt += key > T;
      eq += key == T;
    }
  }
#pragma unroll
  for (int o = 16; o; o >>= 1) {
    gt += __shfl_xor_sync(0xffffffffu, gt, o);
    eq += __shfl_xor_sync(0xffffffffu, eq, o);
  }
  if ((threadIdx.x & 31) == 0) {
    atomicAdd(&s_gt, gt);
    atomicAdd(&s_eq, eq);
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    blk_gt[blockIdx.x] = s_gt;
    blk_eq[blockIdx.x] = s_eq;
  }
}

// Pass B: exclusive scan of the block counts (single block; sequential over chunks of 1024).
__global__ void __launch_bounds__(1024)
select_scan_kernel(const uint32_t* __restrict__ blk_gt, const uint32_t* __restrict__ blk_eq, int64_t nblocks,
                   unsigned long long* __restrict__ off_gt, unsigned long long* __restrict__ off_eq) {
  __shared__ unsigned long long sg[1024], se[1024];
  __shared__ unsigned long long carry_g, carry_e;
  if (threadIdx.x == 0) carry_g = carry_e = 0ull;
  __syncthreads();
  for (int64_t base = 0; base < nblocks; base += 1024) {
    const int64_t i = base + threadIdx.x;
    const unsigned long long g = i < nblocks ? blk_gt[i] : 0ull;
    const unsigned long long e = i < nblocks ? blk_eq[i] : 0ull;
    sg[threadIdx.x] = g;
    se[threadIdx.x] = e;
    __syncthreads();
    for (int o = 1; o < 1024; o <<= 1) {
      unsigned long long ag = 0, ae = 0;
      if (threadIdx.x >= o) {
        ag = sg[threadIdx.x - o];
        ae = se[threadIdx.x - o];
      }
      __syncthreads();
      sg[threadIdx.x] += ag;
      se[threadIdx.x] += ae;
      __syncthreads();
    }
    if (i < nblocks) {
      off_gt[i] = carry_g + sg[threadIdx.x] - g;
      off_eq[i] = carry_e + se[threadIdx.x] - e;
    }
    __syncthreads();
    if (threadIdx.x == 1023) {
      carry_g += sg[1023];
      carry_e += se[1023];
    }
    __syncthreads();
  }
}

// Pass C: ordered write.  Element i is selected if key > T, or key == T and fewer than `need`
// equal keys precede it; its output slot is (#greater before i) + min(#equal before i, need).
// Within a block, thread t owns the kSelItems consecutive elements starting at
// block_base + t*kSelItems, so a scan over threads is a scan over indices.
__global__ void __launch_bounds__(kSelBlock)
select_write_kernel(const float* __restrict__ scores, int64_t n, const SelectState* st,
                    const unsigned long long* __restrict__ off_gt, const unsigned long long* __restrict__ off_eq,
                    int64_t* __restrict__ idx_out, int64_t k) {
  __shared__ uint32_t wg[kSelBlock / 32], we[kSelBlock / 32];
  const uint32_t T = st->threshold;
  const unsigned long long need = st->need_equal;
  const int64_t first = static_cast<int64_t>(blockIdx.x) * kSelTile + static_cast<int64_t>(threadIdx.x) * kSelItems;
  uint32_t keys[kSelItems];
  uint32_t gt = 0, eq = 0;
  int32_t dummy = 0;
#pragma unroll
  for (int t = 0; t < kSelItems; ++t) {
    const int64_t i = first + t;
    keys[t] = i < n ? score_key(scores[i], &dummy) : 0u;
    if (i < n) {
      gt += keys[t] > T;
      eq += keys[t] == T;
    }
  }
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  uint32_t ig = gt, ie = eq;   // inclusive warp scan
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t a = __shfl_up_sync(0xffffffffu, ig, o), b = __shfl_up_sync(0xffffffffu, ie, o);
    if (lane >= o) {
      ig += a;
      ie += b;
    }
  }
  if (lane == 31) {
    wg[warp] = ig;
    we[warp] = ie;
  }
  __syncthreads();
  uint32_t pg = 0, pe = 0;
  for (int w = 0; w < warp; ++w) {
    pg += wg[w];
    pe += we[w];
  }
  unsigned long long cg = off_gt[blockIdx.x] + pg + (ig - gt);
  unsigned long long ce = off_eq[blockIdx.x] + pe + (ie - eq);
#pragma unroll
  for (int t = 0; t < kSelItems; ++t) {
    const int64_t i = first + t;
    if (i < n) {
      const bool g = keys[t] > T, e = keys[t] == T;
      if (g || (e && ce < need)) {
        const unsigned long long slot = cg + (ce < need ? ce : need);
        if (slot < static_cast<unsigned long long>(k)) idx_out[slot] = i;
      }
      cg += g;
      ce += e;
    }
  }
}

}  // namespace szo

// The selection proper, shared by both entry points: four radix passes on the float bits, per-block
// counts, their scan, the ordered write; then the NaN flag is read back (synchronises the stream).
// Every word of scratch that is read has been written by an earlier kernel of this sequence.
static szo_status run_select(const float* scores, int64_t n, int64_t k, int64_t* idx_out, szo::SelectState* state,
                             uint32_t* blk_gt, uint32_t* blk_eq, unsigned long long* off_gt, unsigned long long* off_eq,
                             int64_t nblocks, cudaStream_t st) {
  using namespace szo;
  select_init_kernel<<<1, 256, 0, st>>>(state, static_cast<unsigned long long>(k));
  int64_t hist_blocks = ceil_div(n, kSelBlock * 8);
  if (hist_blocks > 148 * 8) hist_blocks = 148 * 8;
  for (int shift = 24; shift >= 0; shift -= 8) {
    select_hist_kernel<<<static_cast<unsigned>(hist_blocks), kSelBlock, 0, st>>>(scores, n, shift, state);
    select_pick_kernel<<<1, 32, 0, st>>>(state, shift);
  }
  select_count_kernel<<<static_cast<unsigned>(nblocks), kSelBlock, 0, st>>>(scores, n, state, blk_gt, blk_eq);
  select_scan_kernel<<<1, 1024, 0, st>>>(blk_gt, blk_eq, nblocks, off_gt, off_eq);
  select_write_kernel<<<static_cast<unsigned>(nblocks), kSelBlock, 0, st>>>(scores, n, state, off_gt, off_eq,
                                                                          idx_out, k);
  count_launch(12);
  SZO_CHECK_LAUNCH("select_mask kernels");
  int32_t nan_flag = 0;
  SZO_CHECK_CUDA(cudaMemcpyAsync(&nan_flag, &state->nan_flag, sizeof(int32_t), cudaMemcpyDeviceToHost, st));
  SZO_CHECK_CUDA(cudaStreamSynchronize(st));
  SZO_REQUIRE(nan_flag == 0, SZO_ERR_NONFINITE, "scores contain NaN");
  return SZO_OK;
}

extern "C" szo_status szo_select_mask(const float* scores, int64_t n, int64_t k, int64_t* idx_out,
                                      void* workspace, size_t* workspace_bytes, void* stream) {
  using namespace szo;
  SZO_REQUIRE(workspace_bytes != nullptr, SZO_ERR_INVALID_ARG, "workspace_bytes is NULL");
  SZO_REQUIRE(n >= 0 && k >= 0 && k <= n, SZO_ERR_INVALID_ARG, "need 0 <= k <= n (k=%lld, n=%lld)",
              (long long)k, (long long)n);
  const int64_t nblocks = ceil_div(n > 0 ? n : 1, kSelTile);
  const size_t state_bytes = round_up(sizeof(SelectState), 256);
  const size_t cnt_bytes = round_up(static_cast<size_t>(nblocks) * sizeof(uint32_t), 256);
  const size_t off_bytes = round_up(static_cast<size_t>(nblocks) * sizeof(unsigned long long), 256);
  const size_t need = state_bytes + 2 * cnt_bytes + 2 * off_bytes;
  if (workspace == nullptr) {
    *workspace_bytes = need;
    return SZO_OK;
  }
  SZO_REQUIRE(*workspace_bytes >= need, SZO_ERR_WORKSPACE, "workspace too small: %zu < %zu", *workspace_bytes, need);
  SZO_REQUIRE(aligned16(workspace), SZO_ERR_ALIGNMENT, "workspace must be 16-byte aligned");
  if (k == 0) return SZO_OK;
  SZO_REQUIRE(scores && idx_out, SZO_ERR_INVALID_ARG, "NULL pointer");
  SZO_REQUIRE(aligned16(scores) && aligned16(idx_out), SZO_ERR_ALIGNMENT, "buffers must be 16-byte aligned");
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  char* ws = static_cast<char*>(workspace);
  SelectState* state = reinterpret_cast<SelectState*>(ws);
  uint32_t* blk_gt = reinterpret_cast<uint32_t*>(ws + state_bytes);
  uint32_t* blk_eq = reinterpret_cast<uint32_t*>(ws + state_bytes + cnt_bytes);
  unsigned long long* off_gt = reinterpret_cast<unsigned long long*>(ws + state_bytes + 2 * cnt_bytes);
  unsigned long long* off_eq = reinterpret_cast<unsigned long long*>(ws + state_bytes + 2 * cnt_bytes + off_bytes);

  return run_select(scores, n, k, idx_out, state, blk_gt, blk_eq, off_gt, off_eq, nblocks, st);
}


// ------------------------------------------------------------------------------ no-allocation variant
// Same selection with the scratch memory held inside the library image instead of a caller
// workspace.  kStaticSelectMaxN bounds the size: 2^26 scores need 8192 blocks of per-block counts
// and offsets next to the selection state.
namespace szo {
constexpr int64_t kStaticSelectMaxN = int64_t(1) << 26;
constexpr size_t kStaticStateBytes = (sizeof(SelectState) + 255) / 256 * 256;
constexpr size_t kStaticBlocks = static_cast<size_t>(kStaticSelectMaxN / kSelTile);
constexpr size_t kStaticScratchBytes =
    kStaticStateBytes + 2 * kStaticBlocks * sizeof(uint32_t) + 2 * kStaticBlocks * sizeof(unsigned long long);
static __device__ __align__(256) unsigned char g_select_scratch[kStaticScratchBytes];

// Device address of g_select_scratch on the current device, looked up once per device.  In host
// code the symbol name is only a handle; the address a kernel can use comes from
// cudaGetSymbolAddress, with the device that will run the kernels current.  The cached address
// belongs to the device's primary context and is valid as long as that context lives (a
// cudaDeviceReset in the same process would make it stale).
static szo_status static_scratch_address(unsigned char** out) {
  static unsigned char* cached[64] = {nullptr};
  static std::mutex mu;
  std::lock_guard<std::mutex> lock(mu);
  int dev = 0;
  SZO_CHECK_CUDA(cudaGetDevice(&dev));
  SZO_REQUIRE(dev >= 0 && dev < 64, SZO_ERR_UNSUPPORTED, "device ordinal %d not supported", dev);
  if (cached[dev] == nullptr) {
    unsigned char* ptr = nullptr;
    SZO_CHECK_CUDA(cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_select_scratch));
    SZO_REQUIRE(ptr != nullptr, SZO_ERR_CUDA, "cudaGetSymbolAddress returned a null address");
    cached[dev] = ptr;
  }
  *out = cached[dev];
  return SZO_OK;
}
}  // namespace szo

extern "C" szo_status szo_select_mask_static(const float* scores, int64_t n, int64_t k, int64_t* idx_out,
                                             void* stream) {
  using namespace szo;
  SZO_REQUIRE(n >= 0 && k >= 0 && k <= n, SZO_ERR_INVALID_ARG, "need 0 <= k <= n (k=%lld, n=%lld)",
              (long long)k, (long long)n);
  SZO_REQUIRE(n <= kStaticSelectMaxN, SZO_ERR_WORKSPACE,
              "n = %lld exceeds the built-in scratch of szo_select_mask_static (at most %lld scores); "
              "use szo_select_mask with a caller workspace",
              (long long)n, (long long)kStaticSelectMaxN);
  if (k == 0) return SZO_OK;
  SZO_REQUIRE(scores && idx_out, SZO_ERR_INVALID_ARG, "NULL pointer");
  SZO_REQUIRE(aligned16(scores) && aligned16(idx_out), SZO_ERR_ALIGNMENT, "buffers must be 16-byte aligned");
  unsigned char* ws = nullptr;
  SZO_TRY(static_scratch_address(&ws));
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int64_t nblocks = ceil_div(n, kSelTile);
  // fixed carve-up of the array (sized for the maximum), independent of n
  SelectState* state = reinterpret_cast<SelectState*>(ws);
  uint32_t* blk_gt = reinterpret_cast<uint32_t*>(ws + kStaticStateBytes);
  uint32_t* blk_eq = blk_gt + kStaticBlocks;
  unsigned long long* off_gt = reinterpret_cast<unsigned long long*>(blk_eq + kStaticBlocks);
  unsigned long long* off_eq = off_gt + kStaticBlocks;
  // The array keeps whatever the previous call left: the state and histogram are cleared here, the
  // per-block counts and offsets of the nblocks in use are fully overwritten before they are read.
  return run_select(scores, n, k, idx_out, state, blk_gt, blk_eq, off_gt, off_eq, nblocks, st);
}
