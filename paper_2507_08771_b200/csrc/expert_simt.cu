// Expert stage (Eq. 1, Eq. 2 restricted to Union(x), Sec. 3.3), CUDA-core variant.
//
// Two kernels. expert_up: each warp owns 4 neuron rows of one union expert, streams
// their bf16 weights with 128-bit loads, multiplies them with every token of the
// chunk (fp32 FMA, tokens tiled by LT), reduces over the warp, applies Swish and the
// token's router score and stores the fp32 intermediate h[slot][t][j].
// expert_down: each warp owns one output column, runs over all union experts'
// rows of D for that column and over h, reduces, and writes out[t][c] (optionally
// accumulating into an fp32 residual and emitting its bf16 rounding).
// No atomics: every output element has exactly one writer.
#include <mutex>

#include "common.cuh"

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kRows = 4;  // neuron rows per warp task

__device__ __forceinline__ int load_union(const int32_t* union_ids, const int32_t* n_union, int E,
                                          int* ids_sm, uint32_t* status) {
  int nu = *n_union;
  if (nu < 0 || nu > E) {
    if (threadIdx.x == 0) atomicOr(status, BLOCKFFN_DEV_BAD_UNION_COUNT);
    nu = nu < 0 ? 0 : E;
  }
  for (int q = threadIdx.x; q < nu; q += blockDim.x) {
    int id = union_ids[q];
    if (id < 0 || id >= E) {
      atomicOr(status, BLOCKFFN_DEV_BAD_UNION_ID);
      id = -1;
    }
    ids_sm[q] = id;
  }
  __syncthreads();
  return nu;
}

template <int LT>
__global__ void __launch_bounds__(kThreads)
expert_up_simt(const uint16_t* __restrict__ x, const uint16_t* __restrict__ U,
               const float* __restrict__ scores, const int32_t* __restrict__ union_ids,
               const int32_t* __restrict__ n_union, float* __restrict__ h, int L, int d, int E,
               int d_e, int L_max, uint32_t* status) {
  extern __shared__ int ids_sm[];
  const int nu = load_union(union_ids, n_union, E, ids_sm, status);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int groups = d_e / kRows;
  const int tasks = nu * groups;
  const int chunks = d >> 3;
  for (int task = blockIdx.x * kWarps + warp; task < tasks; task += gridDim.x * kWarps) {
    const int q = task / groups, j0 = (task % groups) * kRows;
    const int id = ids_sm[q];
    if (id < 0) continue;
    const uint4* wrow[kRows];
#pragma unroll
    for (int r = 0; r < kRows; ++r)
      wrow[r] = reinterpret_cast<const uint4*>(U + ((size_t)id * d_e + j0 + r) * d);
    for (int t0 = 0; t0 < L; t0 += LT) {
      float acc[kRows][LT];
#pragma unroll
      for (int r = 0; r < kRows; ++r)
#pragma unroll
        for (int t = 0; t < LT; ++t) acc[r][t] = 0.0f;
      for (int c = lane; c < chunks; c += 32) {
        uint4 wv[kRows];
#pragma unroll
        for (int r = 0; r < kRows; ++r) wv[r] = __ldg(wrow[r] + c);
#pragma unroll
        for (int t = 0; t < LT; ++t) {
          if (t0 + t < L) {
            const uint4 xv = __ldg(reinterpret_cast<const uint4*>(x + (size_t)(t0 + t) * d) + c);
            const uint32_t xp[4] = {xv.x, xv.y, xv.z, xv.w};
#pragma unroll
            for (int r = 0; r < kRows; ++r) {
              const uint32_t wp[4] = {wv[r].x, wv[r].y, wv[r].z, wv[r].w};
#pragma unroll
              for (int p = 0; p < 4; ++p) {
                acc[r][t] = fmaf(bf16_lo(wp[p]), bf16_lo(xp[p]), acc[r][t]);
                acc[r][t] = fmaf(bf16_hi(wp[p]), bf16_hi(xp[p]), acc[r][t]);
              }
            }
          }
        }
      }
#pragma unroll
      for (int r = 0; r < kRows; ++r)
#pragma unroll
        for (int t = 0; t < LT; ++t) {
          float v = acc[r][t];
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
          if (lane == r * LT + t && t0 + t < L) {
            const float s = scores[(size_t)(t0 + t) * E + id];
            h[((size_t)q * L_max + t0 + t) * d_e + j0 + r] = s * swish(v);
          }
        }
    }
  }
}

template <int LT>
__global__ void __launch_bounds__(kThreads)
expert_down_simt(const uint16_t* __restrict__ D, const float* __restrict__ h,
                 const int32_t* __restrict__ union_ids, const int32_t* __restrict__ n_union,
                 float* __restrict__ out, uint16_t* __restrict__ x_next, int L, int d, int E,
                 int d_e, int L_max, int accumulate, uint32_t* status) {
  extern __shared__ int ids_sm[];
  const int nu = load_union(union_ids, n_union, E, ids_sm, status);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int K = nu * d_e;
  for (int c = blockIdx.x * kWarps + warp; c < d; c += gridDim.x * kWarps) {
    for (int t0 = 0; t0 < L; t0 += LT) {
      float acc[LT];
#pragma unroll
      for (int t = 0; t < LT; ++t) acc[t] = 0.0f;
      for (int kk = lane * 4; kk < K; kk += 128) {
        const int q = kk / d_e, j = kk - q * d_e;
        const int id = ids_sm[q];
        if (id < 0) continue;
        const uint2 wv = __ldg(reinterpret_cast<const uint2*>(D + ((size_t)id * d + c) * d_e + j));
        const float w0 = bf16_lo(wv.x), w1 = bf16_hi(wv.x), w2 = bf16_lo(wv.y), w3 = bf16_hi(wv.y);
#pragma unroll
        for (int t = 0; t < LT; ++t) {
          if (t0 + t < L) {
            const float4 hv =
                *reinterpret_cast<const float4*>(h + ((size_t)q * L_max + t0 + t) * d_e + j);
            acc[t] = fmaf(hv.x, w0, acc[t]);
            acc[t] = fmaf(hv.y, w1, acc[t]);
            acc[t] = fmaf(hv.z, w2, acc[t]);
            acc[t] = fmaf(hv.w, w3, acc[t]);
          }
        }
      }
#pragma unroll
      for (int t = 0; t < LT; ++t) {
        float v = acc[t];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        if (lane == t && t0 + t < L) {
          const size_t p = (size_t)(t0 + t) * d + c;
          if (accumulate) v += out[p];
          out[p] = v;
          if (x_next) x_next[p] = (uint16_t)f32_to_bf16_bits(v);
        }
      }
    }
  }
}

template <int LT>
cudaError_t launch_lt(blockffn_ctx* c, const blockffn_weights* w, const void* x,
                      const float* scores, int L, const int32_t* union_ids,
                      const int32_t* n_union, float* out, void* x_next, int call_flags,
                      cudaStream_t st) {
  const int E = c->cfg.E, d = c->cfg.d, d_e = c->cfg.d_e;
  const size_t sm = sizeof(int) * (size_t)E;
  const int up_tasks = E * (d_e / kRows);
  int grid_up = (up_tasks + kWarps - 1) / kWarps;
  if (grid_up > c->num_sms * 4) grid_up = c->num_sms * 4;
  int grid_dn = (d + kWarps - 1) / kWarps;
  if (grid_dn > c->num_sms * 4) grid_dn = c->num_sms * 4;
  expert_up_simt<LT><<<grid_up, kThreads, sm, st>>>(
      static_cast<const uint16_t*>(x), static_cast<const uint16_t*>(w->U), scores, union_ids,
      n_union, c->h32, L, d, E, d_e, c->cfg.L_max, c->status);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  expert_down_simt<LT><<<grid_dn, kThreads, sm, st>>>(
      static_cast<const uint16_t*>(w->D), c->h32, union_ids, n_union, out,
      static_cast<uint16_t*>(x_next), L, d, E, d_e, c->cfg.L_max,
      (call_flags & BLOCKFFN_CALL_ACCUMULATE) ? 1 : 0, c->status);
  c->launches += 2;
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_expert_simt(blockffn_ctx* c, const blockffn_weights* w, const void* x,
                               const float* scores, int L, const int32_t* union_ids,
                               const int32_t* n_union, float* out, void* x_next, int call_flags,
                               cudaStream_t st) {
  if (L <= 1) return launch_lt<1>(c, w, x, scores, L, union_ids, n_union, out, x_next, call_flags, st);
  if (L <= 2) return launch_lt<2>(c, w, x, scores, L, union_ids, n_union, out, x_next, call_flags, st);
  if (L <= 4) return launch_lt<4>(c, w, x, scores, L, union_ids, n_union, out, x_next, call_flags, st);
  return launch_lt<8>(c, w, x, scores, L, union_ids, n_union, out, x_next, call_flags, st);
}

// ---- expert stage without a handle and without any allocation ---------------------------
//
// Scratch for blockffn_expert_ffn_noalloc: the fp32 intermediate h[q][t][j] of the two
// CUDA-core kernels above, preceded by a 256-byte header whose first word is the status word
// those kernels want. The array is part of the library image: every GPU that loads the
// library holds these bytes until the process exits.
#define BLOCKFFN_NOALLOC_HEADER 256
static __device__ __align__(256) unsigned char
    g_noalloc_scratch[BLOCKFFN_NOALLOC_HEADER + BLOCKFFN_NOALLOC_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
// Device address of g_noalloc_scratch per device, looked up once per device. In host code
// the array's name is only a handle for the runtime, never an address a kernel may be given.
// The pair (address, SM count) of a device is written and read under the mutex, so that a
// second host thread never sees one without the other.
struct NoallocDevice {
  unsigned char* ptr;
  int sms;
};
NoallocDevice g_noalloc_dev[kMaxDevices] = {};
std::mutex g_noalloc_mutex;
}  // namespace

extern "C" blockffn_status blockffn_expert_ffn_noalloc(
    const blockffn_config* cfg, const blockffn_weights* w, const void* x, const float* scores,
    int32_t L, const int32_t* union_ids, const int32_t* n_union, float* out, void* x_next,
    int32_t call_flags, void* stream) {
  auto bad16 = [](const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; };
  auto bad4 = [](const void* p) { return (reinterpret_cast<uintptr_t>(p) & 3u) != 0; };
  if (!cfg || !w || !w->U || !w->D || !x || !scores || !union_ids || !n_union || !out)
    return BLOCKFFN_ERR_INVALID_ARG;
  if (cfg->d < 8 || cfg->d_e < 8 || cfg->E < 1 || L < 1) return BLOCKFFN_ERR_INVALID_ARG;
  if (cfg->d % 8 || cfg->d_e % 8 || cfg->E > 1024 || L > 32 || cfg->d > (1 << 20) ||
      cfg->d_e > (1 << 16))
    return BLOCKFFN_ERR_UNSUPPORTED;
  // the intermediate of this call must fit the fixed scratch
  if ((size_t)cfg->E * (size_t)L * (size_t)cfg->d_e * sizeof(float) >
      (size_t)BLOCKFFN_NOALLOC_SCRATCH_BYTES)
    return BLOCKFFN_ERR_WORKSPACE;
  if (bad16(w->U) || bad16(w->D) || bad16(x) || bad16(out) || bad16(x_next) || bad4(scores) ||
      bad4(union_ids) || bad4(n_union) || x_next == x)
    return BLOCKFFN_ERR_INVALID_ARG;
  if (call_flags & ~(BLOCKFFN_CALL_ACCUMULATE | BLOCKFFN_CALL_INDEPENDENT | BLOCKFFN_CALL_INDEPENDENT_X))
    return BLOCKFFN_ERR_INVALID_ARG;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return BLOCKFFN_ERR_CUDA;
  NoallocDevice nd;
  {
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    if (!g_noalloc_dev[dev].ptr) {   // first call on this device, with this device current
      unsigned char* ptr = nullptr;
      int sms = 0;
      if (cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_noalloc_scratch) != cudaSuccess ||
          !ptr ||
          cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
        cudaGetLastError();
        return BLOCKFFN_ERR_CUDA;
      }
      g_noalloc_dev[dev].sms = sms;
      g_noalloc_dev[dev].ptr = ptr;
    }
    nd = g_noalloc_dev[dev];
  }
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // The status word is shared by all calls and keeps its last value: start it at zero.
  if (cudaMemsetAsync(nd.ptr, 0, BLOCKFFN_NOALLOC_HEADER, st) != cudaSuccess)
    return BLOCKFFN_ERR_CUDA;
  blockffn_ctx tmp{};          // a view for the launcher: nothing in it owns memory
  tmp.cfg = *cfg;
  tmp.cfg.L_max = L;           // h is laid out [q][L][d_e]
  tmp.device = dev;
  tmp.num_sms = nd.sms;
  tmp.words = (cfg->E + 31) / 32;
  tmp.status = reinterpret_cast<uint32_t*>(nd.ptr);
  tmp.h32 = reinterpret_cast<float*>(nd.ptr + BLOCKFFN_NOALLOC_HEADER);
  const cudaError_t e =
      launch_expert_simt(&tmp, w, x, scores, L, union_ids, n_union, out, x_next, call_flags, st);
  return e == cudaSuccess ? BLOCKFFN_OK : BLOCKFFN_ERR_CUDA;
}
