// RegTop-k sparsification step for N workers batched on one B200 (sm_100a): kernels and C ABI.
//
// One round (regtopk_worker_step + regtopk_aggregate) is this chain of kernels on one stream:
//
//   k_sample_cutoff   per worker: read a strided sample of a = eps + g, pick a candidate cutoff key
//                     from the sample's order statistics (a guess that only has to be low enough)
//   k_stream          the one Theta(N*d) pass: a = eps + g written in place over eps, every entry
//                     whose key bits(|a|) reaches the cutoff appended to the worker's candidate list
//   k_override        the <= k entries of the previous mask's support: posterior distortion,
//                     tanh regulariser, regularised score (Algorithm 2 steps 8-9)
//   k_select          per worker: exact radix select of the k largest (score, lowest index) among
//                     candidates + overrides; winners are set in a bitmask
//   k_dense_select    only for a worker whose cutoff guess was too high or whose list overflowed:
//                     exact radix select over the whole row (slow, always right)
//   k_select (again)  takes over the winners of the dense path
//   k_emit            ordered walk of the bitmask: ascending (index, a[index]) pairs, residual zeroed
//   k_aggregate       server sum in worker order, clearing last round's entries first
//
// The selection key of an entry is the bit pattern of its non-negative binary32 score, which orders
// like the score; the 64-bit composite (key << 32 | ~index) orders like (score descending, index
// ascending) and is unique per entry, so "the k largest composites" is the mask with the
// lowest-index tie rule and needs no further tie handling.
//
// Off the previous support the score is |a| itself (regulariser exactly 1), so no score array is
// ever written: the accumulator that has to be stored anyway is the only dense output.
//
// All floating-point steps use the round-to-nearest intrinsics, which the compiler never contracts
// into fused multiply-adds.

#include <cuda_runtime.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#include <math.h>

#include "regtopk.h"

namespace {

typedef unsigned long long u64;
typedef uint32_t u32;

constexpr int kTileWords = 2048;           // bitmask words per emission tile
constexpr int kTileShift = 16;             // log2(coordinates per tile) = log2(2048 * 32)
constexpr int kSampleSectors = 4096;       // 32-byte sectors sampled per worker
constexpr int kSampleMax = kSampleSectors * 8;
constexpr int kBlockSel = 1024;            // threads of the per-worker kernels
constexpr int kStreamThreads = 256;
constexpr int kWarpList = 256;             // per-warp staging list of k_stream (entries)
constexpr u32 kFull = 0xFFFFFFFFu;

enum : u32 { kStateNormal = 0, kStateNeedDense = 1, kStateDenseDone = 2 };
enum : u32 { kErrCountMismatch = 1u, kErrDenseSelect = 2u };

struct WorkerCtl {
  u32 cutoff;      // candidate cutoff key of this round
  u32 cand_count;  // entries appended (may exceed the capacity: then the list overflowed)
  u32 state;       // kState*
  u32 n_valid;     // valid items seen by the select (diagnostics)
};

struct GlobalCtl {
  u32 err;
  u32 pad;
  u64 dense_workers;
};

__device__ __forceinline__ u64 make_composite(u32 key, u32 idx) {
  return (static_cast<u64>(key) << 32) | static_cast<u64>(kFull - idx);
}
__device__ __forceinline__ u32 composite_idx(u64 c) { return kFull - static_cast<u32>(c); }

// ---------------------------------------------------------------------------------------------
// block-wide helpers (blockDim.x a multiple of 32, at most 1024)
// ---------------------------------------------------------------------------------------------

// Exclusive prefix sum of v over the block in thread order; *total receives the block sum.
// s_scan: 33 words of shared memory.  Every thread of the block must call it.
__device__ __forceinline__ u32 block_excl_scan(u32 v, u32* s_scan, u32* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
  u32 inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    u32 t = __shfl_up_sync(kFull, inc, o);
    if (lane >= o) inc += t;
  }
  if (lane == 31) s_scan[warp] = inc;
  __syncthreads();
  if (warp == 0) {
    u32 w = lane < nwarps ? s_scan[lane] : 0u;
    u32 winc = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      u32 t = __shfl_up_sync(kFull, winc, o);
      if (lane >= o) winc += t;
    }
    s_scan[lane] = winc - w;
    if (lane == 31) s_scan[32] = winc;
  }
  __syncthreads();
  u32 res = inc - v + s_scan[warp];
  *total = s_scan[32];
  __syncthreads();
  return res;
}

// In a histogram of nbins (a multiple of blockDim.x or smaller than it), find the bin that holds the
// r-th entry counted from the top bin down (r >= 1).  s_res[0] = bin (or 0xFFFFFFFF if the
// histogram holds fewer than r entries), s_res[1] = entries in bins above it, s_res[2] = total.
__device__ __forceinline__ void block_find_from_top(const u32* hist, int nbins, u32 r, u32* s_scan,
                                                    u32* s_res) {
  const int per = nbins >= (int)blockDim.x ? nbins / (int)blockDim.x : 1;
  const int first = (int)threadIdx.x * per;  // position counted from the top
  u32 sum = 0;
  if (first < nbins) {
    for (int i = 0; i < per; ++i) sum += hist[nbins - 1 - (first + i)];
  }
  if (threadIdx.x == 0) s_res[0] = kFull;
  u32 total;
  u32 excl = block_excl_scan(sum, s_scan, &total);  // contains __syncthreads
  if (first < nbins && excl < r && r <= excl + sum) {
    u32 acc = excl;
    for (int i = 0; i < per; ++i) {
      u32 h = hist[nbins - 1 - (first + i)];
      if (acc + h >= r) {
        s_res[0] = (u32)(nbins - 1 - (first + i));
        s_res[1] = acc;
        break;
      }
      acc += h;
    }
  }
  if (threadIdx.x == 0) s_res[2] = total;
  __syncthreads();
}

// Warp-aggregated reservation in a shared counter: returns this lane's slot if pred, any value if not.
__device__ __forceinline__ u32 warp_reserve(bool pred, u32* s_counter) {
  const u32 m = __ballot_sync(kFull, pred);
  if (m == 0) return 0;
  const int lane = threadIdx.x & 31;
  const int leader = __ffs(m) - 1;
  u32 base = 0;
  if (lane == leader) base = atomicAdd(s_counter, (u32)__popc(m));
  base = __shfl_sync(kFull, base, leader);
  return base + (u32)__popc(m & ((1u << lane) - 1u));
}

// ---------------------------------------------------------------------------------------------
// tanh(x), x >= 0, as a fixed sequence of individually rounded binary32 operations:
//   x >= 9.25 -> 1;   x < 0.25 -> x + x*q with the odd Taylor terms up to x^9;
//   else (1 - t)/(1 + t), t = exp(-2x) = 2^n * P(f), y = (-2x)*log2(e), n = rint(y), f = y - n,
//   P = degree-7 Taylor polynomial of 2^f (Horner).
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ float tanh_fixed(float x) {
  if (x >= 9.25f) return 1.0f;
  if (x < 0.25f) {
    const float x2 = __fmul_rn(x, x);
    float q = __fadd_rn(__uint_as_float(0xbd5d0dd1u), __fmul_rn(x2, __uint_as_float(0x3cb327a4u)));
    q = __fadd_rn(__uint_as_float(0x3e088889u), __fmul_rn(x2, q));
    q = __fadd_rn(__uint_as_float(0xbeaaaaabu), __fmul_rn(x2, q));
    q = __fmul_rn(x2, q);
    return __fadd_rn(x, __fmul_rn(x, q));
  }
  const float y = __fmul_rn(__fmul_rn(-2.0f, x), __uint_as_float(0x3fb8aa3bu));
  const float n = rintf(y);
  const float f = __fsub_rn(y, n);
  float p = __fadd_rn(__uint_as_float(0x39218489u), __fmul_rn(f, __uint_as_float(0x377fe5feu)));
  p = __fadd_rn(__uint_as_float(0x3aaec3ffu), __fmul_rn(f, p));
  p = __fadd_rn(__uint_as_float(0x3c1d955bu), __fmul_rn(f, p));
  p = __fadd_rn(__uint_as_float(0x3d635847u), __fmul_rn(f, p));
  p = __fadd_rn(__uint_as_float(0x3e75fdf0u), __fmul_rn(f, p));
  p = __fadd_rn(__uint_as_float(0x3f317218u), __fmul_rn(f, p));
  p = __fadd_rn(1.0f, __fmul_rn(f, p));
  // n is in [-27, -1] on this branch, so 2^n is a normal number and the product is exact
  const float scale = __uint_as_float((u32)((int)n + 127) << 23);
  const float t = __fmul_rn(p, scale);
  return __fdiv_rn(__fsub_rn(1.0f, t), __fadd_rn(1.0f, t));
}

template <bool BF16>
__device__ __forceinline__ float load_grad(const void* row, int64_t j) {
  if (BF16) {
    return __uint_as_float((u32)__ldg(static_cast<const unsigned short*>(row) + j) << 16);
  } else {
    return __ldg(static_cast<const float*>(row) + j);
  }
}

// ---------------------------------------------------------------------------------------------
// k_sample_cutoff: one block per worker.
// ---------------------------------------------------------------------------------------------
struct SampleArgs {
  const void* grads;
  int64_t grad_ld;
  const float* eps;
  int64_t ld;
  int64_t d;
  int64_t k_target;  // entries the cutoff should leave above it (k, or 2k when overrides can demote)
  WorkerCtl* ctl;
  GlobalCtl* gctl;
  u32* tcount;
  int ntiles;
  int force_dense;
};

template <bool BF16>
__global__ void __launch_bounds__(kBlockSel) k_sample_cutoff(SampleArgs p) {
  extern __shared__ u32 s_dyn[];
  u32* s_keys = s_dyn;               // kSampleMax
  u32* s_hist = s_dyn + kSampleMax;  // 4096
  __shared__ u32 s_scan[33];
  __shared__ u32 s_res[3];
  const int n = blockIdx.x;
  const int tid = threadIdx.x;

  for (int t = tid; t < p.ntiles; t += blockDim.x) p.tcount[(size_t)n * p.ntiles + t] = 0;
  if (p.force_dense) {
    if (tid == 0) {
      p.ctl[n].cutoff = kFull;  // no key reaches it: the stream pass collects nothing
      p.ctl[n].cand_count = 0;
      p.ctl[n].state = kStateNeedDense;
      p.ctl[n].n_valid = 0;
      atomicAdd(&p.gctl->dense_workers, 1ull);
    }
    return;
  }

  const int64_t Q = (p.d + 7) >> 3;  // 8-element sectors in the row
  const bool all = Q <= kSampleSectors;
  const int nsect = all ? (int)Q : kSampleSectors;
  const int M = all ? (int)p.d : kSampleMax;  // samples that lie inside the row
  const float* eps_row = p.eps + (size_t)n * p.ld;
  const char* grow = static_cast<const char*>(p.grads) + (size_t)n * p.grad_ld * (BF16 ? 2 : 4);

  for (int i = tid; i < 4096; i += blockDim.x) s_hist[i] = 0;
  __syncthreads();
  for (int i = tid; i < nsect * 8; i += blockDim.x) {
    const int s = i >> 3, e = i & 7;
    const int64_t q = all ? s : (int64_t)(((u64)s * (u64)Q) / (u64)kSampleSectors);
    const int64_t j = q * 8 + e;
    u32 key = 0;
    if (j < p.d) {
      const float a = __fadd_rn(eps_row[j], load_grad<BF16>(grow, j));
      key = __float_as_uint(a) & 0x7FFFFFFFu;
      atomicAdd(&s_hist[key >> 19], 1u);
    }
    s_keys[i] = key;
  }
  __syncthreads();

  // rank to read off the sample: expected sample count above the target quantile plus a margin of
  // four standard deviations (the count is close to Poisson) and a constant
  u32 r;
  {
    const double lam = (double)p.k_target * (double)M / (double)p.d;
    double rr = (M == p.d) ? (double)p.k_target : ceil(lam + 4.0 * sqrt(lam) + 8.0);
    r = rr > (double)M ? (u32)M + 1u : (u32)rr;
  }
  u32 cutoff = 0;
  if (r <= (u32)M) {
    block_find_from_top(s_hist, 4096, r, s_scan, s_res);
    const u32 b1 = s_res[0], above1 = s_res[1];
    __syncthreads();
    if (b1 != kFull) {
      for (int i = tid; i < 1024; i += blockDim.x) s_hist[i] = 0;
      __syncthreads();
      for (int i = tid; i < nsect * 8; i += blockDim.x) {
        const u32 key = s_keys[i];
        if ((key >> 19) == b1) {
          // out-of-row sample slots hold key 0 and were not counted in level 1; keep them out
          const int s = i >> 3, e = i & 7;
          const int64_t q = all ? s : (int64_t)(((u64)s * (u64)Q) / (u64)kSampleSectors);
          if (q * 8 + e < p.d) atomicAdd(&s_hist[(key >> 9) & 1023u], 1u);
        }
      }
      __syncthreads();
      block_find_from_top(s_hist, 1024, r - above1, s_scan, s_res);
      const u32 b2 = s_res[0];
      cutoff = (b1 << 19) | ((b2 == kFull ? 0u : b2) << 9);
    }
  }
  if (tid == 0) {
    p.ctl[n].cutoff = cutoff;
    p.ctl[n].cand_count = 0;
    p.ctl[n].state = kStateNormal;
    p.ctl[n].n_valid = 0;
  }
}

// ---------------------------------------------------------------------------------------------
// k_stream: a = eps + g for all workers, in place; candidates appended.  Persistent grid, one
// warp per 512-element chunk, chunks dealt round-robin so that neighbouring warps read
// neighbouring memory.  12 (fp32) or 10 (bf16) bytes of HBM traffic per coordinate.
// ---------------------------------------------------------------------------------------------
struct StreamArgs {
  const void* grads;
  int64_t grad_ld;
  float* eps;
  int64_t ld;
  int64_t d;
  int N;
  WorkerCtl* ctl;
  u64* cand;       // [N][stride]
  int64_t cap;     // entries of a row the stream pass may fill
  int64_t stride;
};

__device__ __forceinline__ void stream_flush(u64* list, u32& wcount, WorkerCtl* ctl, u64* cand,
                                             int64_t cap, int lane) {
  __syncwarp();
  if (wcount) {
    u32 base = 0;
    if (lane == 0) base = atomicAdd(&ctl->cand_count, wcount);
    base = __shfl_sync(kFull, base, 0);
    for (u32 i = lane; i < wcount; i += 32) {
      const u64 pos = (u64)base + i;
      if (pos < (u64)cap) cand[pos] = list[i];
    }
  }
  wcount = 0;
  __syncwarp();
}

template <bool BF16, bool VEC>
__global__ void __launch_bounds__(kStreamThreads) k_stream(StreamArgs p) {
  __shared__ u64 s_list[kStreamThreads / 32][kWarpList];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  u64* list = s_list[warp];
  u32 wcount = 0;  // warp-uniform
  const int64_t chunks_per_row = (p.d + 511) >> 9;
  const int64_t total = chunks_per_row * p.N;
  const int64_t nwarps = (int64_t)gridDim.x * (kStreamThreads / 32);
  int cur_n = -1;
  u32 cutoff = kFull;
  float* eps_row = nullptr;
  const char* grow = nullptr;

  for (int64_t c = (int64_t)blockIdx.x * (kStreamThreads / 32) + warp; c < total; c += nwarps) {
    const int n = (int)(c / chunks_per_row);
    const int64_t base = (c - (int64_t)n * chunks_per_row) << 9;
    if (n != cur_n) {
      if (cur_n >= 0) stream_flush(list, wcount, p.ctl + cur_n, p.cand + (size_t)cur_n * p.stride, p.cap, lane);
      cur_n = n;
      cutoff = p.ctl[n].cutoff;
      eps_row = p.eps + (size_t)n * p.ld;
      grow = static_cast<const char*>(p.grads) + (size_t)n * p.grad_ld * (BF16 ? 2 : 4);
    }
    const bool full = base + 512 <= p.d;  // warp-uniform
    float4 e[4], g[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int64_t j = base + u * 128 + lane * 4;
      e[u] = __ldcs(reinterpret_cast<const float4*>(eps_row + j));  // rows are padded: in bounds
      if (VEC && (full || j + 3 < p.d)) {
        if (BF16) {
          const uint2 raw = __ldcs(reinterpret_cast<const uint2*>(grow + j * 2));
          g[u].x = __uint_as_float(raw.x << 16);
          g[u].y = __uint_as_float(raw.x & 0xFFFF0000u);
          g[u].z = __uint_as_float(raw.y << 16);
          g[u].w = __uint_as_float(raw.y & 0xFFFF0000u);
        } else {
          g[u] = __ldcs(reinterpret_cast<const float4*>(grow + j * 4));
        }
      } else {
        g[u].x = (j + 0 < p.d) ? load_grad<BF16>(grow, j + 0) : 0.0f;
        g[u].y = (j + 1 < p.d) ? load_grad<BF16>(grow, j + 1) : 0.0f;
        g[u].z = (j + 2 < p.d) ? load_grad<BF16>(grow, j + 2) : 0.0f;
        g[u].w = (j + 3 < p.d) ? load_grad<BF16>(grow, j + 3) : 0.0f;
      }
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int64_t j = base + u * 128 + lane * 4;
      float4 a;
      a.x = __fadd_rn(e[u].x, g[u].x);
      a.y = __fadd_rn(e[u].y, g[u].y);
      a.z = __fadd_rn(e[u].z, g[u].z);
      a.w = __fadd_rn(e[u].w, g[u].w);
      *reinterpret_cast<float4*>(eps_row + j) = a;  // padding receives 0 + 0
      const u32 k0 = __float_as_uint(a.x) & 0x7FFFFFFFu, k1 = __float_as_uint(a.y) & 0x7FFFFFFFu;
      const u32 k2 = __float_as_uint(a.z) & 0x7FFFFFFFu, k3 = __float_as_uint(a.w) & 0x7FFFFFFFu;
      const bool h0 = k0 >= cutoff && (full || j + 0 < p.d);
      const bool h1 = k1 >= cutoff && (full || j + 1 < p.d);
      const bool h2 = k2 >= cutoff && (full || j + 2 < p.d);
      const bool h3 = k3 >= cutoff && (full || j + 3 < p.d);
      if (__any_sync(kFull, h0 | h1 | h2 | h3)) {
        const u32 lt = (1u << lane) - 1u;
        u32 m;
        m = __ballot_sync(kFull, h0);
        if (h0) list[wcount + __popc(m & lt)] = make_composite(k0, (u32)j);
        wcount += __popc(m);
        m = __ballot_sync(kFull, h1);
        if (h1) list[wcount + __popc(m & lt)] = make_composite(k1, (u32)j + 1);
        wcount += __popc(m);
        m = __ballot_sync(kFull, h2);
        if (h2) list[wcount + __popc(m & lt)] = make_composite(k2, (u32)j + 2);
        wcount += __popc(m);
        m = __ballot_sync(kFull, h3);
        if (h3) list[wcount + __popc(m & lt)] = make_composite(k3, (u32)j + 3);
        wcount += __popc(m);
        if (wcount >= kWarpList - 128)  // the next step adds at most 128
          stream_flush(list, wcount, p.ctl + cur_n, p.cand + (size_t)cur_n * p.stride, p.cap, lane);
      }
    }
  }
  if (cur_n >= 0) stream_flush(list, wcount, p.ctl + cur_n, p.cand + (size_t)cur_n * p.stride, p.cap, lane);
}

// ---------------------------------------------------------------------------------------------
// k_override: regularised scores on the previous support (Eq. (Delta_def), Algorithm 2 step 9).
// ---------------------------------------------------------------------------------------------
struct OverrideArgs {
  const float* eps;  // holds a after k_stream
  int64_t ld;
  const float* g_prev;
  const int32_t* prev_idx;
  const float* prev_val;
  const float* omega;
  float mu;
  int64_t k;
  int N;
  const WorkerCtl* ctl;
  u32* ovr_key;   // [N][k] score bits of every previous-support entry
  u64* ovr_comp;  // [N][k] composite if the score reaches the cutoff, else 0
};

__global__ void __launch_bounds__(256) k_override(OverrideArgs p) {
  const int64_t total = p.k * p.N;
  for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < total;
       t += (int64_t)gridDim.x * blockDim.x) {
    const int n = (int)(t / p.k);
    const int32_t j = p.prev_idx[t];
    const float ap = p.prev_val[t];
    const float G = p.g_prev[j];
    const float a = p.eps[(size_t)n * p.ld + j];
    const float w = p.omega[n];
    const float num = __fsub_rn(G, __fmul_rn(w, ap));
    const float den = __fmul_rn(w, a);
    float m = 1.0f;
    if (den != 0.0f) {
      const float delta = __fdiv_rn(num, den);
      const float r = fabsf(__fadd_rn(1.0f, delta));
      m = tanh_fixed(__fdiv_rn(r, p.mu));
    }
    const u32 key = __float_as_uint(__fmul_rn(fabsf(a), m));
    p.ovr_key[t] = key;
    p.ovr_comp[t] = key >= p.ctl[n].cutoff ? make_composite(key, (u32)j) : 0ull;
  }
}

// ---------------------------------------------------------------------------------------------
// k_select: one block per worker; exact k largest composites among candidates and overrides.
// ---------------------------------------------------------------------------------------------
struct SelectArgs {
  WorkerCtl* ctl;
  GlobalCtl* gctl;
  u64* candA;        // [N][stride]; the stream pass fills at most capA entries of a row
  int64_t capA;
  u64* candB;        // [N][stride]
  int64_t stride;    // capA + k: what one histogram bin can hold (all candidates plus all overrides)
  const u64* ovr_comp;
  const int32_t* prev_idx;
  u32* bitmask;      // [N][W]
  int64_t W;
  u32* tcount;       // [N][ntiles]
  u32* toff;         // [N][ntiles]
  int ntiles;
  int64_t k;
  int use_marks;     // previous support carries regularised scores (round >= 1, mu > 0)
  int has_prev;      // bitmask holds last round's mask, to be cleared
  int phase;         // 0: normal workers; 1: workers finished by the dense path
};

__device__ __forceinline__ void set_winner(const SelectArgs& p, int n, u32 idx) {
  atomicOr(&p.bitmask[(size_t)n * p.W + (idx >> 5)], 1u << (idx & 31));
  atomicAdd(&p.tcount[(size_t)n * p.ntiles + (idx >> kTileShift)], 1u);
}

__global__ void __launch_bounds__(kBlockSel) k_select(SelectArgs p) {
  __shared__ u32 s_hist[4096];
  __shared__ u32 s_scan[33];
  __shared__ u32 s_res[3];
  __shared__ u32 s_cnt;
  const int n = blockIdx.x, tid = threadIdx.x;
  WorkerCtl* ctl = p.ctl + n;
  const u32 state = ctl->state;
  if (p.phase == 0 ? state != kStateNormal : state != kStateDenseDone) return;

  u64* A = p.candA + (size_t)n * p.stride;
  u64* B = p.candB + (size_t)n * p.stride;
  const u64* O = p.ovr_comp + (size_t)n * p.k;
  const int32_t* prev_idx = p.prev_idx + (size_t)n * p.k;
  u32* mask = p.bitmask + (size_t)n * p.W;
  const u32 cand_count = ctl->cand_count;
  const bool dense_done = p.phase == 1;
  const bool use_marks = p.use_marks && !dense_done;
  const u32 ncand = (u64)cand_count <= (u64)p.capA ? cand_count : (u32)p.capA;
  const u32 novr = use_marks ? (u32)p.k : 0u;
  const u32 k = (u32)p.k;

  u32 need = k;
  u32 nsrc = 0;
  if (!dense_done) {
    // filter: drop candidates that lie on the previous support (their score is the override's),
    // histogram the top 12 key bits of everything valid
    for (int i = tid; i < 4096; i += blockDim.x) s_hist[i] = 0;
    __syncthreads();
    for (u32 i = tid; i < ncand; i += blockDim.x) {
      u64 c = A[i];
      if (use_marks) {
        const u32 idx = composite_idx(c);
        if ((mask[idx >> 5] >> (idx & 31)) & 1u) {
          A[i] = 0ull;
          continue;
        }
      }
      atomicAdd(&s_hist[(u32)(c >> 51)], 1u);
    }
    for (u32 i = tid; i < novr; i += blockDim.x) {
      const u64 c = O[i];
      if (c) atomicAdd(&s_hist[(u32)(c >> 51)], 1u);
    }
    __syncthreads();
    block_find_from_top(s_hist, 4096, k, s_scan, s_res);
    const u32 b1 = s_res[0], above1 = s_res[1], nvalid = s_res[2];
    __syncthreads();
    if (b1 == kFull || (u64)cand_count > (u64)p.capA) {
      // too few valid candidates (cutoff guessed too high) or the list overflowed: dense path
      if (tid == 0) {
        ctl->state = kStateNeedDense;
        ctl->n_valid = nvalid;
        atomicAdd(&p.gctl->dense_workers, 1ull);
      }
      return;
    }
    if (tid == 0) {
      ctl->n_valid = nvalid;
      s_cnt = 0;
    }
    // every probe of the old mask is done: clear it (whole words; all their bits are old marks)
    if (p.has_prev)
      for (u32 i = tid; i < k; i += blockDim.x) mask[(u32)prev_idx[i] >> 5] = 0u;
    __syncthreads();
    // classify: above the bin -> winner; inside the bin -> list B for refinement
    const u32 iters = (ncand + novr + blockDim.x - 1) / blockDim.x;
    for (u32 it = 0; it < iters; ++it) {
      const u32 i = it * blockDim.x + tid;
      u64 c = 0ull;
      if (i < ncand) c = A[i];
      else if (i < ncand + novr) c = O[i - ncand];
      const u32 bin = (u32)(c >> 51);
      if (c && bin > b1) set_winner(p, n, composite_idx(c));
      const bool inbin = c && bin == b1;
      const u32 pos = warp_reserve(inbin, &s_cnt);
      if (inbin) B[pos] = c;
    }
    __syncthreads();
    need = k - above1;
    nsrc = s_cnt;
    __syncthreads();
  } else {
    // the dense path left exactly k winners in A
    if (p.has_prev)
      for (u32 i = tid; i < k; i += blockDim.x) mask[(u32)prev_idx[i] >> 5] = 0u;
    __syncthreads();
    need = k;
    nsrc = k;
    u64* t = A; A = B; B = t;  // so that "src" below is the list with the winners
  }

  // refinement on the remaining 51 composite bits, 8 at a time; src/dst ping-pong between B and A
  u64* src = B;
  u64* dst = A;
  int shift = 43;
  while (true) {
    if (need == 0) break;
    if (need == nsrc) {
      for (u32 i = tid; i < nsrc; i += blockDim.x) set_winner(p, n, composite_idx(src[i]));
      break;
    }
    if (shift < -8) {  // all 51 bits consumed and still undecided: composites were not unique
      if (tid == 0) atomicOr(&p.gctl->err, kErrCountMismatch);
      break;
    }
    const int sh = shift >= 0 ? shift : 0;
    const u32 dmask = shift >= 0 ? 255u : 7u;  // the last digit is the low 3 bits
    for (int i = tid; i < 256; i += blockDim.x) s_hist[i] = 0;
    if (tid == 0) s_cnt = 0;
    __syncthreads();
    for (u32 i = tid; i < nsrc; i += blockDim.x) atomicAdd(&s_hist[(u32)(src[i] >> sh) & dmask], 1u);
    __syncthreads();
    block_find_from_top(s_hist, 256, need, s_scan, s_res);
    const u32 b = s_res[0], above = s_res[1];
    __syncthreads();
    if (b == kFull) {  // cannot happen: need <= nsrc
      if (tid == 0) atomicOr(&p.gctl->err, kErrCountMismatch);
      break;
    }
    const u32 iters = (nsrc + blockDim.x - 1) / blockDim.x;
    for (u32 it = 0; it < iters; ++it) {
      const u32 i = it * blockDim.x + tid;
      u64 c = 0ull;
      u32 dg = 0;
      if (i < nsrc) {
        c = src[i];
        dg = (u32)(c >> sh) & dmask;
        if (dg > b) set_winner(p, n, composite_idx(c));
      }
      const bool inbin = i < nsrc && dg == b;
      const u32 pos = warp_reserve(inbin, &s_cnt);
      if (inbin) dst[pos] = c;
    }
    __syncthreads();
    need -= above;
    nsrc = s_cnt;
    __syncthreads();
    u64* t = src; src = dst; dst = t;
    shift -= 8;
  }
  __syncthreads();
  __threadfence_block();

  // exclusive scan of the per-tile winner counts -> output offsets of k_emit
  {
    u32* tc = p.tcount + (size_t)n * p.ntiles;
    u32* to = p.toff + (size_t)n * p.ntiles;
    const int per = (p.ntiles + blockDim.x - 1) / blockDim.x;
    const int first = tid * per;
    u32 sum = 0;
    for (int i = 0; i < per; ++i)
      if (first + i < p.ntiles) sum += __ldcg(tc + first + i);
    u32 total;
    u32 run = block_excl_scan(sum, s_scan, &total);
    for (int i = 0; i < per; ++i)
      if (first + i < p.ntiles) {
        to[first + i] = run;
        run += __ldcg(tc + first + i);
      }
    if (tid == 0 && total != k) atomicOr(&p.gctl->err, kErrCountMismatch);
  }
}

// ---------------------------------------------------------------------------------------------
// k_dense_select: exact selection over the whole row for workers in state NeedDense.  One block per
// worker; slow (every pass walks d entries with 1024 threads) but right for any input, including
// rows of equal values.  Leaves the k winners in the worker's candidate list A.
// ---------------------------------------------------------------------------------------------
struct DenseArgs {
  WorkerCtl* ctl;
  GlobalCtl* gctl;
  const float* eps;  // holds a
  int64_t ld;
  int64_t d;
  int64_t k;
  const u32* bitmask;
  int64_t W;
  const int32_t* prev_idx;
  const u32* ovr_key;
  u64* candA;
  int64_t stride;
  int use_marks;
};

__device__ __forceinline__ u32 dense_key(const DenseArgs& p, int n, int64_t j) {
  if (p.use_marks) {
    const u32 w = p.bitmask[(size_t)n * p.W + (j >> 5)];
    if ((w >> (j & 31)) & 1u) {
      const int32_t* pi = p.prev_idx + (size_t)n * p.k;
      int64_t lo = 0, hi = p.k;
      while (lo < hi) {
        const int64_t mid = (lo + hi) >> 1;
        if (pi[mid] < (int32_t)j) lo = mid + 1; else hi = mid;
      }
      return p.ovr_key[(size_t)n * p.k + lo];
    }
  }
  return __float_as_uint(p.eps[(size_t)n * p.ld + j]) & 0x7FFFFFFFu;
}

__global__ void __launch_bounds__(kBlockSel) k_dense_select(DenseArgs p) {
  __shared__ u32 s_hist[4096];
  __shared__ u32 s_scan[33];
  __shared__ u32 s_res[3];
  __shared__ u32 s_cnt;
  const int n = blockIdx.x, tid = threadIdx.x;
  WorkerCtl* ctl = p.ctl + n;
  if (ctl->state != kStateNeedDense) return;
  u64* A = p.candA + (size_t)n * p.stride;

  u32 need = (u32)p.k;
  u32 prefix = 0;
  // three digits of the 31-bit key: bits 30..19, 18..7, 6..0
  const int shifts[3] = {19, 7, 0};
  const int widths[3] = {12, 12, 7};
  for (int lv = 0; lv < 3; ++lv) {
    const int sh = shifts[lv], nb = 1 << widths[lv];
    for (int i = tid; i < nb; i += blockDim.x) s_hist[i] = 0;
    __syncthreads();
    for (int64_t j = tid; j < p.d; j += blockDim.x) {
      const u32 key = dense_key(p, n, j);
      if (lv == 0 || (key >> (sh + widths[lv])) == prefix) atomicAdd(&s_hist[(key >> sh) & (nb - 1)], 1u);
    }
    __syncthreads();
    block_find_from_top(s_hist, nb, need, s_scan, s_res);
    const u32 b = s_res[0], above = s_res[1];
    __syncthreads();
    if (b == kFull) {
      if (tid == 0) atomicOr(&p.gctl->err, kErrDenseSelect);
      return;
    }
    need -= above;
    prefix = (prefix << widths[lv]) | b;
  }
  const u32 T = prefix;                   // key of the k-th largest score
  const u32 n_gt = (u32)p.k - need;       // entries strictly above it; `need` ties are to be taken
  if (tid == 0) s_cnt = 0;
  __syncthreads();
  // entries above T, in any order
  for (int64_t base = 0; base < p.d; base += blockDim.x) {
    const int64_t j = base + tid;
    u32 key = 0;
    bool gt = false;
    if (j < p.d) {
      key = dense_key(p, n, j);
      gt = key > T;
    }
    const u32 pos = warp_reserve(gt, &s_cnt);
    if (gt && pos < n_gt) A[pos] = make_composite(key, (u32)j);
  }
  __syncthreads();
  if (tid == 0 && s_cnt != n_gt) atomicOr(&p.gctl->err, kErrDenseSelect);
  // ties in index order: the first `need` of them
  u32 taken = 0;
  for (int64_t base = 0; base < p.d && taken < need; base += blockDim.x) {
    const int64_t j = base + tid;
    const bool tie = j < p.d && dense_key(p, n, j) == T;
    u32 total;
    const u32 rank = taken + block_excl_scan(tie ? 1u : 0u, s_scan, &total);
    if (tie && rank < need) A[n_gt + rank] = make_composite(T, (u32)j);
    taken += total;
  }
  if (tid == 0) {
    if (taken < need) atomicOr(&p.gctl->err, kErrDenseSelect);
    ctl->cand_count = (u32)p.k;
    ctl->state = kStateDenseDone;
  }
}

// ---------------------------------------------------------------------------------------------
// k_emit: ordered walk of the winner bitmask.  One block per (tile, worker); ascending indices.
// ---------------------------------------------------------------------------------------------
struct EmitArgs {
  const u32* bitmask;
  int64_t W;
  const u32* tcount;
  const u32* toff;
  int ntiles;
  float* eps;
  int64_t ld;
  int64_t k;
  int32_t* out_idx;
  float* out_val;
  int32_t* cur_idx;
  float* cur_val;
};

__global__ void __launch_bounds__(256) k_emit(EmitArgs p) {
  __shared__ u32 s_scan[33];
  const int t = blockIdx.x, n = blockIdx.y, tid = threadIdx.x;
  if (p.tcount[(size_t)n * p.ntiles + t] == 0) return;
  const u32* words = p.bitmask + (size_t)n * p.W + (size_t)t * kTileWords + tid * 8;
  const uint4 w0 = *reinterpret_cast<const uint4*>(words);
  const uint4 w1 = *reinterpret_cast<const uint4*>(words + 4);
  u32 w[8] = {w0.x, w0.y, w0.z, w0.w, w1.x, w1.y, w1.z, w1.w};
  u32 c = 0;
#pragma unroll
  for (int i = 0; i < 8; ++i) c += __popc(w[i]);
  u32 total;
  u32 pos = p.toff[(size_t)n * p.ntiles + t] + block_excl_scan(c, s_scan, &total);
  if (c == 0) return;
  float* eps_row = p.eps + (size_t)n * p.ld;
  const size_t obase = (size_t)n * p.k;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    u32 bits = w[i];
    const u32 jbase = ((u32)t * kTileWords + tid * 8 + i) << 5;
    while (bits) {
      const int b = __ffs(bits) - 1;
      bits &= bits - 1;
      const u32 j = jbase + b;
      const float v = eps_row[j];
      eps_row[j] = 0.0f;  // a - a
      if (pos < (u32)p.k) {  // always true when the tile counts are consistent
        p.out_idx[obase + pos] = (int32_t)j;
        p.out_val[obase + pos] = v;
        p.cur_idx[obase + pos] = (int32_t)j;
        p.cur_val[obase + pos] = v;
      }
      ++pos;
    }
  }
}

// ---------------------------------------------------------------------------------------------
// k_aggregate: g = sum_n omega_n * ghat_n in worker order.  The coordinate range is cut into
// gridDim.x slices; a block owns a slice, so all updates of one coordinate happen in one block,
// ordered by the barrier between workers.  Last round's entries are cleared first.
// ---------------------------------------------------------------------------------------------
struct AggArgs {
  float* g;
  int64_t d;
  int N;
  int64_t k;
  const int32_t* cur_idx;
  const float* cur_val;
  const int32_t* prev_idx;
  const float* omega;
  int has_prev;
};

__device__ __forceinline__ int64_t lower_bound_i32(const int32_t* a, int64_t n, int64_t v) {
  int64_t lo = 0, hi = n;
  while (lo < hi) {
    const int64_t mid = (lo + hi) >> 1;
    if ((int64_t)a[mid] < v) lo = mid + 1; else hi = mid;
  }
  return lo;
}

__global__ void __launch_bounds__(256) k_aggregate(AggArgs p) {
  extern __shared__ int64_t s_bounds[];  // [2 lists][N][2]
  const int tid = threadIdx.x;
  const int64_t lo = (int64_t)(((u64)blockIdx.x * (u64)p.d) / gridDim.x);
  const int64_t hi = (int64_t)(((u64)(blockIdx.x + 1) * (u64)p.d) / gridDim.x);
  for (int t = tid; t < 4 * p.N; t += blockDim.x) {
    const int list = t / (2 * p.N), n = (t >> 1) % p.N, side = t & 1;
    const int32_t* arr = (list ? p.prev_idx : p.cur_idx) + (size_t)n * p.k;
    s_bounds[t] = (list && !p.has_prev) ? 0 : lower_bound_i32(arr, p.k, side ? hi : lo);
  }
  __syncthreads();
  if (p.has_prev) {
    for (int n = 0; n < p.N; ++n) {
      const int64_t b = s_bounds[2 * p.N + 2 * n], e = s_bounds[2 * p.N + 2 * n + 1];
      const int32_t* pi = p.prev_idx + (size_t)n * p.k;
      for (int64_t i = b + tid; i < e; i += blockDim.x) p.g[pi[i]] = 0.0f;
    }
    __syncthreads();
  }
  for (int n = 0; n < p.N; ++n) {
    const int64_t b = s_bounds[2 * n], e = s_bounds[2 * n + 1];
    const int32_t* ci = p.cur_idx + (size_t)n * p.k;
    const float* cv = p.cur_val + (size_t)n * p.k;
    const float w = p.omega[n];
    for (int64_t i = b + tid; i < e; i += blockDim.x) {
      const int32_t j = ci[i];
      p.g[j] = __fadd_rn(p.g[j], __fmul_rn(w, cv[i]));
    }
    __syncthreads();
  }
}

// ---------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------
inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct Layout {
  int64_t ld, W, capA, capB;
  int ntiles;
  size_t off_eps, off_g, off_mask, off_tcount, off_toff, off_idx[2], off_val[2], off_ovr_key,
      off_ovr_comp, off_candA, off_candB, off_ctl, off_gctl, off_omega, off_stage_g, off_stage_idx,
      off_stage_val, zero_end, total;
};

bool valid_problem(int64_t d, int32_t N, int64_t k, const regtopk_params* pr) {
  if (!pr) return false;
  if (d < 1 || d > 2147483646LL || N < 1 || N > 65535 || k < 1 || k > d) return false;
  if (!(pr->mu >= 0.0f) || !isfinite(pr->mu)) return false;
  if (pr->grad_dtype != REGTOPK_GRAD_F32 && pr->grad_dtype != REGTOPK_GRAD_BF16) return false;
  if (pr->omega)
    for (int n = 0; n < N; ++n)
      if (!isfinite(pr->omega[n])) return false;
  return true;
}

Layout make_layout(int64_t d, int32_t N, int64_t k, const regtopk_params* pr) {
  Layout L;
  L.ld = (int64_t)align_up((size_t)d, 1024);
  L.ntiles = (int)((d + (1 << kTileShift) - 1) >> kTileShift);
  L.W = (int64_t)L.ntiles * kTileWords;
  const int64_t M = d < kSampleMax ? d : kSampleMax;
  const int64_t kt = pr->mu > 0.0f ? (2 * k < d ? 2 * k : d) : k;
  int64_t cap = 2 * kt + 64 * ((d + M - 1) / M) + 4096;
  if (cap > d) cap = d;
  if (cap < k) cap = k;
  L.capA = cap;
  L.capB = cap + k;
  size_t o = 0;
  auto take = [&](size_t bytes) { size_t at = o; o = align_up(o + bytes, 256); return at; };
  // state that creation and reset clear to zero comes first
  L.off_eps = take((size_t)N * L.ld * 4);
  L.off_g = take(align_up((size_t)d, 64) * 4);
  L.off_mask = take((size_t)N * L.W * 4);
  L.off_tcount = take((size_t)N * L.ntiles * 4);
  L.off_toff = take((size_t)N * L.ntiles * 4);
  L.off_ctl = take((size_t)N * sizeof(WorkerCtl));
  L.off_gctl = take(sizeof(GlobalCtl));
  L.zero_end = o;
  for (int i = 0; i < 2; ++i) {
    L.off_idx[i] = take((size_t)N * k * 4);
    L.off_val[i] = take((size_t)N * k * 4);
  }
  L.off_ovr_key = take((size_t)N * k * 4);
  L.off_ovr_comp = take((size_t)N * k * 8);
  L.off_candA = take((size_t)N * L.capB * 8);
  L.off_candB = take((size_t)N * L.capB * 8);
  L.off_omega = take((size_t)N * 4);
  L.off_stage_g = L.off_stage_idx = L.off_stage_val = 0;
  if (pr->flags & REGTOPK_FLAG_HOST_STAGING) {
    L.off_stage_g = take((size_t)N * L.ld * (pr->grad_dtype == REGTOPK_GRAD_BF16 ? 2 : 4));
    L.off_stage_idx = take((size_t)N * k * 4);
    L.off_stage_val = take((size_t)N * k * 4);
  }
  L.total = o;
  return L;
}

constexpr int kMaxProfile = 4096;

}  // namespace

struct regtopk_ctx {
  int64_t d, k;
  int32_t N;
  float mu;
  int32_t grad_dtype, flags;
  Layout L;
  char* ws;
  cudaStream_t stream;
  int cur;           // which pair buffer receives this round's pairs
  int64_t round;
  int stepped;       // worker_step done, aggregate pending
  int sticky;        // first CUDA error seen
  int num_sms;
  int stream_blocks[4];
  int64_t launches;
  int profiling;
  int n_events;
  cudaEvent_t* ev0;
  cudaEvent_t* ev1;
};

namespace {

template <typename T>
T* at(regtopk_ctx* c, size_t off) { return reinterpret_cast<T*>(c->ws + off); }

int note_cuda(regtopk_ctx* c, cudaError_t e) {
  if (e == cudaSuccess) return REGTOPK_OK;
  if (c && !c->sticky) c->sticky = REGTOPK_ERR_CUDA;
  return REGTOPK_ERR_CUDA;
}

int after_launch(regtopk_ctx* c) {
  c->launches++;
  return note_cuda(c, cudaGetLastError());
}

size_t sample_smem() { return (size_t)(kSampleMax + 4096) * sizeof(u32); }

template <bool BF16, bool VEC>
void launch_stream(regtopk_ctx* c, const StreamArgs& a, int variant) {
  if (c->stream_blocks[variant] == 0) {
    int per_sm = 0;
    cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_stream<BF16, VEC>, kStreamThreads, 0);
    if (per_sm < 1) per_sm = 1;
    c->stream_blocks[variant] = per_sm * c->num_sms;
  }
  const int64_t chunks = ((a.d + 511) >> 9) * a.N;
  int64_t blocks = (chunks + (kStreamThreads / 32) - 1) / (kStreamThreads / 32);
  if (blocks > c->stream_blocks[variant]) blocks = c->stream_blocks[variant];
  k_stream<BF16, VEC><<<(unsigned)blocks, kStreamThreads, 0, c->stream>>>(a);
}

}  // namespace

extern "C" {

const char* regtopk_strerror(int code) {
  switch (code) {
    case REGTOPK_OK: return "ok";
    case REGTOPK_ERR_INVALID_ARG: return "invalid argument";
    case REGTOPK_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case REGTOPK_ERR_SEQUENCE: return "calls out of order (worker_step and aggregate must alternate)";
    case REGTOPK_ERR_CUDA: return "CUDA runtime error";
    case REGTOPK_ERR_INTERNAL: return "device reported an inconsistent selection";
    case REGTOPK_ERR_NO_DEVICE: return "no usable sm_100 device";
    default: return "unknown error code";
  }
}

size_t regtopk_workspace_bytes(int64_t d, int32_t N, int64_t k, const regtopk_params* params) {
  if (!valid_problem(d, N, k, params)) return 0;
  return make_layout(d, N, k, params).total;
}

int regtopk_state_reset(regtopk_ctx* c) {
  if (!c) return REGTOPK_ERR_INVALID_ARG;
  int rc = note_cuda(c, cudaMemsetAsync(c->ws, 0, c->L.zero_end, c->stream));
  c->round = 0;
  c->stepped = 0;
  c->cur = 0;
  return rc;
}

int regtopk_create(regtopk_ctx** out, int64_t d, int32_t N, int64_t k, const regtopk_params* params,
                   void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (!out) return REGTOPK_ERR_INVALID_ARG;
  *out = nullptr;
  if (!valid_problem(d, N, k, params) || !workspace) return REGTOPK_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(workspace) % 256 != 0) return REGTOPK_ERR_INVALID_ARG;
  Layout L = make_layout(d, N, k, params);
  if (workspace_bytes < L.total) return REGTOPK_ERR_WORKSPACE_TOO_SMALL;
  int dev = 0, major = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return REGTOPK_ERR_NO_DEVICE;
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess ||
      major != 10)
    return REGTOPK_ERR_NO_DEVICE;
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (cudaFuncSetAttribute(k_sample_cutoff<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           (int)sample_smem()) != cudaSuccess ||
      cudaFuncSetAttribute(k_sample_cutoff<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           (int)sample_smem()) != cudaSuccess) {
    cudaGetLastError();
    return REGTOPK_ERR_NO_DEVICE;
  }
  regtopk_ctx* c = static_cast<regtopk_ctx*>(calloc(1, sizeof(regtopk_ctx)));
  if (!c) return REGTOPK_ERR_INVALID_ARG;
  c->d = d; c->k = k; c->N = N;
  c->mu = params->mu;
  c->grad_dtype = params->grad_dtype;
  c->flags = params->flags;
  c->L = L;
  c->ws = static_cast<char*>(workspace);
  c->stream = static_cast<cudaStream_t>(cuda_stream);
  c->num_sms = sms > 0 ? sms : 148;
  float* om = static_cast<float*>(malloc(sizeof(float) * N));
  if (!om) { free(c); return REGTOPK_ERR_INVALID_ARG; }
  for (int n = 0; n < N; ++n) om[n] = params->omega ? params->omega[n] : 1.0f / (float)N;
  int rc = regtopk_state_reset(c);
  // pageable source: the copy is staged before the call returns, so om may be freed right away
  if (rc == REGTOPK_OK)
    rc = note_cuda(c, cudaMemcpyAsync(c->ws + L.off_omega, om, sizeof(float) * N,
                                      cudaMemcpyHostToDevice, c->stream));
  if (rc == REGTOPK_OK) rc = note_cuda(c, cudaStreamSynchronize(c->stream));
  free(om);
  if (rc != REGTOPK_OK) { free(c); return rc; }
  *out = c;
  return REGTOPK_OK;
}

int regtopk_worker_step(regtopk_ctx* c, const void* grads, int64_t grad_ld, int32_t* out_idx,
                        float* out_val) {
  if (!c || !grads || !out_idx || !out_val || grad_ld < c->d) return REGTOPK_ERR_INVALID_ARG;
  if (c->stepped) return REGTOPK_ERR_SEQUENCE;
  const Layout& L = c->L;
  const bool bf16 = c->grad_dtype == REGTOPK_GRAD_BF16;
  const bool has_prev = c->round >= 1;
  const bool use_marks = has_prev && c->mu > 0.0f;
  const int prev = c->cur ^ 1;
  const uintptr_t gaddr = reinterpret_cast<uintptr_t>(grads);
  const bool vec = (grad_ld % 4 == 0) && (gaddr % (bf16 ? 8 : 16) == 0);
  int rc = REGTOPK_OK;

  SampleArgs sa;
  sa.grads = grads; sa.grad_ld = grad_ld; sa.eps = at<float>(c, L.off_eps); sa.ld = L.ld; sa.d = c->d;
  sa.k_target = use_marks ? (2 * c->k < c->d ? 2 * c->k : c->d) : c->k;
  sa.ctl = at<WorkerCtl>(c, L.off_ctl); sa.gctl = at<GlobalCtl>(c, L.off_gctl);
  sa.tcount = at<u32>(c, L.off_tcount); sa.ntiles = L.ntiles;
  sa.force_dense = (c->flags & REGTOPK_FLAG_FORCE_DENSE_SELECT) ? 1 : 0;
  if (bf16) k_sample_cutoff<true><<<c->N, kBlockSel, sample_smem(), c->stream>>>(sa);
  else k_sample_cutoff<false><<<c->N, kBlockSel, sample_smem(), c->stream>>>(sa);
  if ((rc = after_launch(c))) return rc;

  StreamArgs st;
  st.grads = grads; st.grad_ld = grad_ld; st.eps = at<float>(c, L.off_eps); st.ld = L.ld; st.d = c->d;
  st.N = c->N; st.ctl = sa.ctl; st.cand = at<u64>(c, L.off_candA); st.cap = L.capA; st.stride = L.capB;
  const bool prof = c->profiling && c->n_events < kMaxProfile;
  if (prof) cudaEventRecord(c->ev0[c->n_events], c->stream);
  if (bf16) { if (vec) launch_stream<true, true>(c, st, 3); else launch_stream<true, false>(c, st, 2); }
  else { if (vec) launch_stream<false, true>(c, st, 1); else launch_stream<false, false>(c, st, 0); }
  if (prof) cudaEventRecord(c->ev1[c->n_events++], c->stream);
  if ((rc = after_launch(c))) return rc;

  if (use_marks) {
    OverrideArgs oa;
    oa.eps = at<float>(c, L.off_eps); oa.ld = L.ld; oa.g_prev = at<float>(c, L.off_g);
    oa.prev_idx = at<int32_t>(c, L.off_idx[prev]); oa.prev_val = at<float>(c, L.off_val[prev]);
    oa.omega = at<float>(c, L.off_omega); oa.mu = c->mu; oa.k = c->k; oa.N = c->N; oa.ctl = sa.ctl;
    oa.ovr_key = at<u32>(c, L.off_ovr_key); oa.ovr_comp = at<u64>(c, L.off_ovr_comp);
    const int64_t total = c->k * c->N;
    int64_t blocks = (total + 255) / 256;
    if (blocks > (int64_t)c->num_sms * 16) blocks = (int64_t)c->num_sms * 16;
    k_override<<<(unsigned)blocks, 256, 0, c->stream>>>(oa);
    if ((rc = after_launch(c))) return rc;
  }

  SelectArgs se;
  se.ctl = sa.ctl; se.gctl = sa.gctl; se.candA = at<u64>(c, L.off_candA); se.capA = L.capA;
  se.candB = at<u64>(c, L.off_candB); se.stride = L.capB; se.ovr_comp = at<u64>(c, L.off_ovr_comp);
  se.prev_idx = at<int32_t>(c, L.off_idx[prev]); se.bitmask = at<u32>(c, L.off_mask); se.W = L.W;
  se.tcount = sa.tcount; se.toff = at<u32>(c, L.off_toff); se.ntiles = L.ntiles; se.k = c->k;
  se.use_marks = use_marks; se.has_prev = has_prev; se.phase = 0;
  k_select<<<c->N, kBlockSel, 0, c->stream>>>(se);
  if ((rc = after_launch(c))) return rc;

  DenseArgs da;
  da.ctl = sa.ctl; da.gctl = sa.gctl; da.eps = at<float>(c, L.off_eps); da.ld = L.ld; da.d = c->d;
  da.k = c->k; da.bitmask = at<u32>(c, L.off_mask); da.W = L.W; da.prev_idx = se.prev_idx;
  da.ovr_key = at<u32>(c, L.off_ovr_key); da.candA = se.candA; da.stride = L.capB; da.use_marks = use_marks;
  k_dense_select<<<c->N, kBlockSel, 0, c->stream>>>(da);
  if ((rc = after_launch(c))) return rc;
  se.phase = 1;
  k_select<<<c->N, kBlockSel, 0, c->stream>>>(se);
  if ((rc = after_launch(c))) return rc;

  EmitArgs em;
  em.bitmask = se.bitmask; em.W = L.W; em.tcount = se.tcount; em.toff = se.toff; em.ntiles = L.ntiles;
  em.eps = at<float>(c, L.off_eps); em.ld = L.ld; em.k = c->k; em.out_idx = out_idx; em.out_val = out_val;
  em.cur_idx = at<int32_t>(c, L.off_idx[c->cur]); em.cur_val = at<float>(c, L.off_val[c->cur]);
  k_emit<<<dim3((unsigned)L.ntiles, (unsigned)c->N), 256, 0, c->stream>>>(em);
  if ((rc = after_launch(c))) return rc;

  c->stepped = 1;
  return REGTOPK_OK;
}

int regtopk_aggregate(regtopk_ctx* c, float* out_g) {
  if (!c) return REGTOPK_ERR_INVALID_ARG;
  if (!c->stepped) return REGTOPK_ERR_SEQUENCE;
  const Layout& L = c->L;
  AggArgs a;
  a.g = at<float>(c, L.off_g); a.d = c->d; a.N = c->N; a.k = c->k;
  a.cur_idx = at<int32_t>(c, L.off_idx[c->cur]); a.cur_val = at<float>(c, L.off_val[c->cur]);
  a.prev_idx = at<int32_t>(c, L.off_idx[c->cur ^ 1]); a.omega = at<float>(c, L.off_omega);
  a.has_prev = c->round >= 1;
  int64_t blocks = (int64_t)c->num_sms * 8;
  if (blocks > c->d) blocks = c->d;
  const size_t smem = (size_t)4 * c->N * sizeof(int64_t);
  k_aggregate<<<(unsigned)blocks, 256, smem, c->stream>>>(a);
  int rc = after_launch(c);
  if (rc) return rc;
  if (out_g)
    rc = note_cuda(c, cudaMemcpyAsync(out_g, a.g, (size_t)c->d * 4, cudaMemcpyDeviceToDevice, c->stream));
  c->cur ^= 1;  // this round's pairs are now "previous"
  c->round++;
  c->stepped = 0;
  return rc;
}

int regtopk_global_gradient(regtopk_ctx* c, const float** dev_ptr) {
  if (!c || !dev_ptr) return REGTOPK_ERR_INVALID_ARG;
  *dev_ptr = at<float>(c, c->L.off_g);
  return REGTOPK_OK;
}

int regtopk_round_host(regtopk_ctx* c, const void* h_grads, int64_t grad_ld, int32_t* h_idx,
                       float* h_val, float* h_g) {
  if (!c || !h_grads || !h_idx || !h_val) return REGTOPK_ERR_INVALID_ARG;
  if (!(c->flags & REGTOPK_FLAG_HOST_STAGING) || grad_ld < c->d || grad_ld > c->L.ld)
    return REGTOPK_ERR_INVALID_ARG;
  const Layout& L = c->L;
  const size_t esz = c->grad_dtype == REGTOPK_GRAD_BF16 ? 2 : 4;
  int rc = note_cuda(c, cudaMemcpyAsync(c->ws + L.off_stage_g, h_grads, (size_t)c->N * grad_ld * esz,
                                        cudaMemcpyHostToDevice, c->stream));
  if (rc) return rc;
  rc = regtopk_worker_step(c, c->ws + L.off_stage_g, grad_ld, at<int32_t>(c, L.off_stage_idx),
                           at<float>(c, L.off_stage_val));
  if (rc) return rc;
  rc = regtopk_aggregate(c, nullptr);
  if (rc) return rc;
  const size_t pb = (size_t)c->N * c->k * 4;
  rc = note_cuda(c, cudaMemcpyAsync(h_idx, c->ws + L.off_stage_idx, pb, cudaMemcpyDeviceToHost, c->stream));
  if (!rc) rc = note_cuda(c, cudaMemcpyAsync(h_val, c->ws + L.off_stage_val, pb, cudaMemcpyDeviceToHost, c->stream));
  if (!rc && h_g)
    rc = note_cuda(c, cudaMemcpyAsync(h_g, c->ws + L.off_g, (size_t)c->d * 4, cudaMemcpyDeviceToHost, c->stream));
  if (!rc) rc = note_cuda(c, cudaStreamSynchronize(c->stream));
  return rc;
}

int regtopk_status(regtopk_ctx* c) {
  if (!c) return REGTOPK_ERR_INVALID_ARG;
  GlobalCtl h;
  memset(&h, 0, sizeof h);
  int rc = note_cuda(c, cudaMemcpyAsync(&h, c->ws + c->L.off_gctl, sizeof h, cudaMemcpyDeviceToHost, c->stream));
  if (!rc) rc = note_cuda(c, cudaStreamSynchronize(c->stream));
  if (c->sticky) return c->sticky;
  if (rc) return rc;
  return h.err ? REGTOPK_ERR_INTERNAL : REGTOPK_OK;
}

int regtopk_get_stats(regtopk_ctx* c, regtopk_stats* out) {
  if (!c || !out) return REGTOPK_ERR_INVALID_ARG;
  GlobalCtl h;
  memset(&h, 0, sizeof h);
  WorkerCtl* w = static_cast<WorkerCtl*>(malloc(sizeof(WorkerCtl) * c->N));
  if (!w) return REGTOPK_ERR_INVALID_ARG;
  int rc = note_cuda(c, cudaMemcpyAsync(&h, c->ws + c->L.off_gctl, sizeof h, cudaMemcpyDeviceToHost, c->stream));
  if (!rc) rc = note_cuda(c, cudaMemcpyAsync(w, c->ws + c->L.off_ctl, sizeof(WorkerCtl) * c->N, cudaMemcpyDeviceToHost, c->stream));
  if (!rc) rc = note_cuda(c, cudaStreamSynchronize(c->stream));
  if (!rc) {
    out->rounds = c->round + (c->stepped ? 1 : 0);
    out->kernel_launches = c->launches;
    out->dense_select_workers = (int64_t)h.dense_workers;
    out->candidates_last = 0;
    for (int n = 0; n < c->N; ++n) out->candidates_last += w[n].cand_count;
    out->candidate_capacity = c->L.capA;
  }
  free(w);
  return rc;
}

int regtopk_profile_enable(regtopk_ctx* c, int enable) {
  if (!c) return REGTOPK_ERR_INVALID_ARG;
  if (enable && !c->ev0) {
    c->ev0 = static_cast<cudaEvent_t*>(calloc(kMaxProfile, sizeof(cudaEvent_t)));
    c->ev1 = static_cast<cudaEvent_t*>(calloc(kMaxProfile, sizeof(cudaEvent_t)));
    if (!c->ev0 || !c->ev1) return REGTOPK_ERR_INVALID_ARG;
    for (int i = 0; i < kMaxProfile; ++i) {
      if (cudaEventCreate(&c->ev0[i]) != cudaSuccess || cudaEventCreate(&c->ev1[i]) != cudaSuccess)
        return note_cuda(c, cudaErrorUnknown);
    }
  }
  c->profiling = enable ? 1 : 0;
  return REGTOPK_OK;
}

int regtopk_profile_read(regtopk_ctx* c, double* stream_kernel_ms, int64_t* calls) {
  if (!c || !stream_kernel_ms || !calls) return REGTOPK_ERR_INVALID_ARG;
  int rc = note_cuda(c, cudaStreamSynchronize(c->stream));
  double sum = 0.0;
  for (int i = 0; i < c->n_events && !rc; ++i) {
    float ms = 0.f;
    rc = note_cuda(c, cudaEventElapsedTime(&ms, c->ev0[i], c->ev1[i]));
    sum += ms;
  }
  *stream_kernel_ms = sum;
  *calls = c->n_events;
  c->n_events = 0;
  return rc;
}

int regtopk_debug_residual(regtopk_ctx* c, const float** dev_ptr, int64_t* ld) {
  if (!c || !dev_ptr || !ld) return REGTOPK_ERR_INVALID_ARG;
  *dev_ptr = at<float>(c, c->L.off_eps);
  *ld = c->L.ld;
  return REGTOPK_OK;
}

int regtopk_destroy(regtopk_ctx* c) {
  if (!c) return REGTOPK_ERR_INVALID_ARG;
  cudaStreamSynchronize(c->stream);
  if (c->ev0) {
    for (int i = 0; i < kMaxProfile; ++i) {
      if (c->ev0[i]) cudaEventDestroy(c->ev0[i]);
      if (c->ev1 && c->ev1[i]) cudaEventDestroy(c->ev1[i]);
    }
  }
  free(c->ev0);
  free(c->ev1);
  free(c);
  return REGTOPK_OK;
}

}  // extern "C"
