// RegTop-k sparsification step for N workers batched on one B200 (sm_100a): kernels and C ABI.
//
// One round (regtopk_worker_step + regtopk_aggregate) is four kernels on one stream, chained with
// programmatic dependent launch:
//
//   k_sample_cutoff   a cluster of 8 blocks per worker reads a strided sample of a = eps + g and
//                     derives, from the sample's order statistics, a candidate cutoff key (a guess that
//                     only has to be low enough) and the bin width the select will use.  Further
//                     clusters of the same launch compute the regularised scores on the previous mask's
//                     support (Eq. (Delta_def), Algorithm 2 steps 8-9) meanwhile.
//   k_stream          the one Theta(N*d) pass: a = eps + g written in place over eps; every entry
//                     whose key bits(|a|) reaches the cutoff and that is not on the previous support is
//                     appended to the worker's candidate list
//   k_post            one thread-block cluster per worker: exact selection of the k largest (score,
//                     lowest index) among candidates and overrides, winners set in a bitmask; per-quad
//                     prefix counts of the bitmask give every winner its rank, and each winner writes
//                     its (index, a[index]) pair there and zeroes its residual.  If the cutoff guess was
//                     too high or the list overflowed, the same cluster runs an exact radix select over
//                     the whole row.
//   k_aggregate       server sum in worker order, one thread per sent pair, ranks looked up through
//                     the prefix counts written during emission
//
// When N*k is large the list phases of k_post run as kernels of their own on the whole grid instead
// (k_wide_hist, k_wide_classify, k_post for the refinement only, k_wide_prefix, k_wide_emit, k_unzip): see
// "Wide mode" below.  regtopk_worker_step_inplace uses a read-only variant of k_stream on rows into which
// the caller has already added the gradients.
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
// into fused multiply-adds.  No kernel waits on another block except through the hardware cluster
// barrier, which every block of a cluster reaches the same number of times.

#include <cooperative_groups.h>
#include <cuda_runtime.h>

#include <atomic>
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#include "regtopk.h"

namespace cg = cooperative_groups;

namespace {

typedef unsigned long long u64;
typedef uint32_t u32;

constexpr int kSampleSectors = 8192;       // 32-byte sectors sampled per worker
constexpr int kSampleMax = kSampleSectors * 8;
constexpr int kBlockSel = 1024;            // threads per block of k_sample_cutoff
#ifndef REGTOPK_POST_THREADS
#define REGTOPK_POST_THREADS 1024
#endif
constexpr int kBlockPost = REGTOPK_POST_THREADS;  // threads per block of k_post
constexpr int kStreamThreads = 256;
constexpr int kWarpList = 256;             // per-warp staging list of k_stream (entries)
constexpr int kCutSpan = 512;              // coordinates per entry of the layer-wise cutoff table (divides every chunk size)
constexpr int kBins = 4096;                // histogram bins of the select
constexpr int kMaxCluster = 16;
constexpr int kMaxSegments = kMaxCluster * 32;  // mask segments per row: one per warp of a k_post cluster
constexpr u32 kFull = 0xFFFFFFFFu;
constexpr u32 kExactRounds = 1024;     // rounds of exact cutoffs after a first fallback to the dense path;
constexpr u32 kExactRoundsMax = 1u << 20;  // doubled after every further one, up to this

// One thread, after its worker fell back to the dense path because the cutoff was off.
__device__ __forceinline__ void ask_for_exact_cutoffs(volatile u32* exact_rounds, volatile u32* exact_window) {
  const u32 w = *exact_window;
  const u32 next = w == 0u ? kExactRounds : (w >= kExactRoundsMax / 2u ? kExactRoundsMax : 2u * w);
  *exact_window = next;
  *exact_rounds = next;
}

enum : u32 { kErrCountMismatch = 1u, kErrDenseSelect = 2u, kErrRefine = 4u, kErrBounds = 8u };

// Checked build (-DREGTOPK_DEBUG=1): every access whose index is computed from data (a candidate's
// index, a rank, a list position) is tested against its array's extent first; an index out of range is
// counted here and the access skipped, and regtopk_status then reports REGTOPK_ERR_INTERNAL.  Nothing
// traps.  The release build compiles the tests away.
#ifndef REGTOPK_DEBUG
#define REGTOPK_DEBUG 0
#endif
#if REGTOPK_DEBUG
__device__ unsigned int g_bounds_faults;
#define RT_INB(cond) ((cond) ? true : (atomicAdd(&g_bounds_faults, 1u), false))
// Gradients must be finite.  The checked build counts the accumulators that are not (infinity or NaN) as the streaming
// pass forms them; regtopk_status then reports REGTOPK_ERR_INVALID_ARG until regtopk_state_reset.
__device__ unsigned int g_nonfinite;
#define RT_NOTE_NONFINITE(key, in) do { if ((in) && (key) > 0x7F7FFFFFu) atomicAdd(&g_nonfinite, 1u); } while (0)
#else
#define RT_INB(cond) true
#define RT_NOTE_NONFINITE(key, in) do { } while (0)
#endif

struct WorkerCtl {
  u32 cutoff;       // candidate cutoff key of this round
  u32 bin_shift;    // select bins: bin = min(kBins - 1, (key - cutoff) >> bin_shift)
  u32 cand_count;   // entries appended by k_stream (may exceed the capacity: the list overflowed)
  u32 force_dense;  // skip the candidate path (testing flag)
  u32 bcount;       // length of the refinement list
  u32 acount;       // dense path: entries above the threshold gathered so far
  u32 n_valid;      // valid items seen by the select (diagnostics)
  u32 b1;           // wide mode: threshold bin, entries above it, and whether the row needs the dense
  u32 above1;       //   exact path (written by k_wide_classify, read by k_post and k_wide_emit)
  u32 go_dense;
  u32 took_dense;   // wide mode: the dense path produced the winner list (written by k_post)
  u32 exact_rounds; // rounds for which k_sample_cutoff resolves the cutoff exactly inside its bin; set when the
                    // selection had to fall back to the dense path, counted down by k_sample_cutoff, and kept
                    // across rounds (nothing else resets it but regtopk_state_reset)
  u32 exact_window; // length of the last such stretch: it doubles with every further fallback
  u32 hint;         // the sampled cutoff of this round, kept for k_dense when the candidate path is not taken (0xFFFFFFFF: none)
  u32 seg_done;     // k_dense: segments of this worker whose first digit has been searched in the current pass; zero between passes
  u32 pad;
};

struct GlobalCtl {
  u32 err;
  u32 dense_flags;    // k_dense: kFlag* bits that all blocks of the launch read after a grid barrier; zero between launches
  u64 dense_workers;
};

// Programmatic dependent launch: every kernel of the round is launched with the stream-serialization
// attribute, lets its successor be scheduled at once (so that the successor's blocks take over SMs as
// this kernel's blocks retire instead of after a full drain and launch), and itself waits here, before
// its first memory access, until its predecessor has completed and its writes are visible.
__device__ __forceinline__ void grid_dependency_begin() {
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

__device__ __forceinline__ u64 make_composite(u32 key, u32 idx) {
  return (static_cast<u64>(key) << 32) | static_cast<u64>(kFull - idx);
}
__device__ __forceinline__ u32 composite_idx(u64 c) { return kFull - static_cast<u32>(c); }

// ---------------------------------------------------------------------------------------------
// block-wide helpers (blockDim.x a multiple of 32, at most 1024)
// ---------------------------------------------------------------------------------------------

// Histogram increment for data that may pile up in one bin (error feedback packs the entries under the
// selection threshold into a narrow band): when all lanes of a warp that have an item hit the same bin, one of
// them adds the count; otherwise every lane adds its own.  Every lane of the warp must call it (pred: this
// lane has an item).
__device__ __forceinline__ void hist_add_aggregated(u32* hist, bool pred, u32 bin) {
  const u32 act = __ballot_sync(kFull, pred);
  if (act == 0u) return;
  const int first = __ffs(act) - 1;
  const u32 bin0 = __shfl_sync(kFull, bin, first);
  if (__all_sync(kFull, !pred || bin == bin0)) {
    if ((int)(threadIdx.x & 31) == first) atomicAdd(&hist[bin0], (u32)__popc(act));
  } else if (pred) {
    atomicAdd(&hist[bin], 1u);
  }
}

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

// m^p for 0 <= m <= 1, p >= 1 (exponent variant of Remark 3), as a fixed sequence of individually
// rounded binary32 operations: 0 -> 0, 1 -> 1, else 2^(p * log2 m); log2 m = e + log2 f with m = 2^e f,
// f in (sqrt(1/2), sqrt 2], ln f = 2 s (1 + s2/3 + s2^2/5 + s2^3/7 + s2^4/9), s = (f - 1)/(f + 1);
// 2^z by the polynomial of tanh_fixed; z < -125 -> 0.
__device__ __forceinline__ float pow_fixed(float m, float p) {
  if (m == 0.0f) return 0.0f;
  if (m >= 1.0f) return 1.0f;
  int e0 = 0;
  if (m < __uint_as_float(0x00800000u)) {  // subnormal: exact scaling into the normal range
    m = __fmul_rn(m, 16777216.0f);
    e0 = -24;
  }
  const u32 b = __float_as_uint(m);
  int e = (int)((b >> 23) & 0xffu) - 127 + e0;
  float f = __uint_as_float((b & 0x7fffffu) | 0x3f800000u);
  if (f > __uint_as_float(0x3fb504f3u)) {  // sqrt(2)
    f = __fmul_rn(f, 0.5f);
    e += 1;
  }
  const float s = __fdiv_rn(__fsub_rn(f, 1.0f), __fadd_rn(f, 1.0f));
  const float s2 = __fmul_rn(s, s);
  float q = __uint_as_float(0x3de38e39u);                                    // 1/9
  q = __fadd_rn(__uint_as_float(0x3e124925u), __fmul_rn(s2, q));             // 1/7
  q = __fadd_rn(__uint_as_float(0x3e4ccccdu), __fmul_rn(s2, q));             // 1/5
  q = __fadd_rn(__uint_as_float(0x3eaaaaabu), __fmul_rn(s2, q));             // 1/3
  q = __fadd_rn(1.0f, __fmul_rn(s2, q));
  const float lnf = __fmul_rn(__fmul_rn(2.0f, s), q);
  const float log2f = __fmul_rn(lnf, __uint_as_float(0x3fb8aa3bu));
  const float L = __fadd_rn((float)e, log2f);
  const float z = __fmul_rn(p, L);
  if (!(z >= -125.0f)) return 0.0f;
  const float n = rintf(z);
  const float fr = __fsub_rn(z, n);
  float P = __fadd_rn(__uint_as_float(0x39218489u), __fmul_rn(fr, __uint_as_float(0x377fe5feu)));
  P = __fadd_rn(__uint_as_float(0x3aaec3ffu), __fmul_rn(fr, P));
  P = __fadd_rn(__uint_as_float(0x3c1d955bu), __fmul_rn(fr, P));
  P = __fadd_rn(__uint_as_float(0x3d635847u), __fmul_rn(fr, P));
  P = __fadd_rn(__uint_as_float(0x3e75fdf0u), __fmul_rn(fr, P));
  P = __fadd_rn(__uint_as_float(0x3f317218u), __fmul_rn(fr, P));
  P = __fadd_rn(1.0f, __fmul_rn(fr, P));
  return __fmul_rn(P, __uint_as_float((u32)((int)n + 127) << 23));  // n in [-125, 0]: exact scaling
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
// k_sample_cutoff: one cluster of kSampleCluster blocks per worker.  Each block gathers its share
// of the sample in one wave of loads and histograms the top 14 key bits (1/64-octave bins); the
// blocks' histograms meet in global memory at the cluster barrier, and the leader reads two order
// statistics off the merged histogram.
// ---------------------------------------------------------------------------------------------
constexpr int kSampleCluster = 8;
constexpr int kSamplePerBlock = kSampleMax / kSampleCluster;  // 8192: eight per thread
constexpr int kSampleBins = 16384;
constexpr int kSampleShift = 17;  // key >> 17: sign-less exponent and six mantissa bits
constexpr int kSamplePadded = kSampleBins + kSampleBins / 16;
__device__ __forceinline__ u32 sample_slot(u32 bin) { return bin + (bin >> 4); }

struct SampleArgs {
  const void* grads;
  int64_t grad_ld;
  const float* eps;
  int64_t ld;
  int64_t d;
  int64_t k;
  int64_t k_target;  // entries the cutoff should leave above it (k, or 2k when overrides can demote)
  WorkerCtl* ctl;
  u32* ghist;  // [N][4][kBins] histograms of k_post, cleared here
  u32* shist;  // [N][kSampleBins] histogram of this kernel; zero on entry (k_post clears it again)
  u32* skeys;  // [N][kSampleMax] the sample's keys (0xFFFFFFFF in unused slots), for the exact second look
  int force_dense;  // 1: no sampling, the dense path is taken; 2: sample, keep the cutoff as a hint, take the dense path
  // Clusters beyond the first N compute the regularised scores of the previous support
  // (Eq. (Delta_def), Algorithm 2 steps 8-9) while the first N sample.  On that support the
  // residual is +0, so the accumulator there is 0 + g.
  int N;
  int use_marks;
  const float* g_prev;
  const int32_t* prev_idx;  // [N][k]
  const float* prev_val;    // [N][k]
  const float* prev_num;    // [N][k] g^{t-1}[j] - omega_n * a^{t-1}[j] per previous pair, formed by k_aggregate while g[j] was
                            // at hand, or NULL (then it is formed here, which costs a gather from g per pair)
  const float* omega;
  float mu;
  float inv_y;              // 1/y of the exponent variant (1: Algorithm 2 as printed)
  u32* ovr_key;             // [N][k] out: score bits
  int share_override;       // the sampling blocks take a share of the override work too
  int inplace;              // the caller has already added g into the rows of eps: a is read from there, grads is NULL
};

// Add a block's histogram to the cluster's in global memory (non-empty bins only).
__device__ __forceinline__ void flush_hist(const u32* s_hist, u32* g_hist, int nbins) {
  for (int i = threadIdx.x; i < nbins; i += blockDim.x) {
    const u32 v = s_hist[i];
    if (v) atomicAdd(&g_hist[i], v);
  }
}

// Regularised scores of the previous support (Eq. (Delta_def), Algorithm 2 steps 8-9) for the items
// first, first + nthreads, ... of the N*k previous pairs; four items per thread in flight.
template <bool BF16>
__device__ __forceinline__ void override_scores(const SampleArgs& p, int64_t first, int64_t nthreads) {
  const int64_t total = p.k * p.N;
  for (int64_t t0 = first; t0 < total; t0 += 4 * nthreads) {
    int32_t j[4];
    float ap[4], G[4], gr[4];
    int wn[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int64_t t = t0 + q * nthreads;
      const bool in = t < total;
      j[q] = in ? p.prev_idx[t] : 0;
      ap[q] = in ? (p.prev_num ? p.prev_num[t] : p.prev_val[t]) : 0.0f;  // with prev_num: the numerator itself
      wn[q] = in ? (int)(t / p.k) : 0;
    }
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const bool in = t0 + q * nthreads < total;
      G[q] = (in && !p.prev_num) ? p.g_prev[j[q]] : 0.0f;
      if (p.inplace)
        gr[q] = in ? p.eps[(size_t)wn[q] * p.ld + j[q]] : 0.0f;  // the residual there was +0: the row holds 0 + g
      else
        gr[q] = in ? load_grad<BF16>(static_cast<const char*>(p.grads) + (size_t)wn[q] * p.grad_ld * (BF16 ? 2 : 4), j[q]) : 0.0f;
    }
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int64_t t = t0 + q * nthreads;
      if (t < total) {
        const float w = p.omega[wn[q]];
        const float a = p.inplace ? gr[q] : __fadd_rn(0.0f, gr[q]);
        const float num = p.prev_num ? ap[q] : __fsub_rn(G[q], __fmul_rn(w, ap[q]));
        const float den = __fmul_rn(w, a);
        float m = 1.0f;
        if (den != 0.0f) {
          const float delta = __fdiv_rn(num, den);
          const float r = fabsf(__fadd_rn(1.0f, delta));
          m = tanh_fixed(__fdiv_rn(r, p.mu));
        }
        if (p.inv_y != 1.0f) m = pow_fixed(m, p.inv_y);  // Remark 3: rank by |a|^y m, i.e. by |a| m^(1/y)
        p.ovr_key[t] = __float_as_uint(__fmul_rn(fabsf(a), m));
      }
    }
  }
}

template <bool BF16>
__global__ void __launch_bounds__(kBlockSel) k_sample_cutoff(SampleArgs p) {
  extern __shared__ u32 s_hist[];  // kSampleBins bins, one pad word after every 16 (bank-conflict-free per-thread runs)
  grid_dependency_begin();
  __shared__ u32 s_scan[33];
  __shared__ u32 s_res[3];
  cg::cluster_group cl = cg::this_cluster();
  const u32 rk = cl.block_rank();
  const int n = blockIdx.x / kSampleCluster;
  const int tid = threadIdx.x;
  if (n >= p.N) {  // an override cluster: no barriers on this path
    if (!p.use_marks) return;
    if (p.share_override)
      override_scores<BF16>(p, (int64_t)blockIdx.x * blockDim.x + tid, (int64_t)gridDim.x * blockDim.x);
    else
      override_scores<BF16>(p, (int64_t)(blockIdx.x - p.N * kSampleCluster) * blockDim.x + tid,
                            (int64_t)(gridDim.x - p.N * kSampleCluster) * blockDim.x);
    return;
  }
  // with many overrides the sampling blocks take their share of them first (the sampling itself is short)
  if (p.use_marks && p.share_override)
    override_scores<BF16>(p, (int64_t)blockIdx.x * blockDim.x + tid, (int64_t)gridDim.x * blockDim.x);
  WorkerCtl* ctl = p.ctl + n;
  u32* shist = p.shist + (size_t)n * kSampleBins;
  // exact cutoff wanted this round (see below)?  Read by every thread of the cluster here, long before the
  // leader's thread 0 counts it down behind the cluster barrier.
  const bool want_exact = ctl->exact_rounds != 0u;

  for (int i = rk * blockDim.x + tid; i < 4 * kBins; i += kSampleCluster * blockDim.x)
    p.ghist[(size_t)n * 4 * kBins + i] = 0;
  if (p.force_dense == 1) {  // the same in every block: nobody reaches a barrier
    if (rk == 0 && tid == 0) {
      ctl->hint = kFull;
      ctl->cutoff = kFull;  // no key reaches it: the stream pass collects nothing
      ctl->bin_shift = 0;
      ctl->cand_count = 0;
      ctl->force_dense = 1;
      ctl->bcount = 0;
      ctl->acount = 0;
      ctl->n_valid = 0;
      ctl->b1 = kFull; ctl->above1 = 0; ctl->go_dense = 0; ctl->took_dense = 0;
    }
    return;
  }

  const int64_t Q = (p.d + 7) >> 3;  // 8-element sectors in the row
  const bool all = Q <= kSampleSectors;
  const int nslots = (all ? (int)Q : kSampleSectors) * 8;
  const int M = all ? (int)p.d : kSampleMax;  // samples that lie inside the row
  const float* eps_row = p.eps + (size_t)n * p.ld;
  const char* grow = static_cast<const char*>(p.grads) + (size_t)n * p.grad_ld * (BF16 ? 2 : 4);

  {  // this block's slots: [rk * kSamplePerBlock, +kSamplePerBlock), eight per thread, one wave of loads
    float e[8], g[8];
    bool ok[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int i = (int)rk * kSamplePerBlock + u * kBlockSel + tid;
      const int sct = i >> 3;
      const int64_t q = all ? sct : (int64_t)(((u64)sct * (u64)Q) / (u64)kSampleSectors);
      const int64_t j = q * 8 + (i & 7);
      ok[u] = i < nslots && j < p.d;
      e[u] = ok[u] ? eps_row[j] : 0.0f;
      g[u] = (ok[u] && !p.inplace) ? load_grad<BF16>(grow, j) : 0.0f;
    }
    for (int i = tid; i < kSamplePadded; i += blockDim.x) s_hist[i] = 0;  // while the loads are in flight
    __syncthreads();
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const u32 key = __float_as_uint(p.inplace ? e[u] : __fadd_rn(e[u], g[u])) & 0x7FFFFFFFu;
      if (want_exact) p.skeys[(size_t)n * kSampleMax + (int)rk * kSamplePerBlock + u * kBlockSel + tid] = ok[u] ? key : kFull;
      if (ok[u]) atomicAdd(&s_hist[sample_slot(key >> kSampleShift)], 1u);
    }
  }
  __syncthreads();
  for (int i = tid; i < kSampleBins; i += blockDim.x) {
    const u32 v = s_hist[sample_slot((u32)i)];
    if (v) atomicAdd(&shist[i], v);
  }
  cl.sync();  // histogram of the whole sample complete
  if (rk != 0) return;
  for (int i = tid; i < kSampleBins; i += blockDim.x) s_hist[sample_slot((u32)i)] = __ldcg(&shist[i]);
  __syncthreads();

  // Ranks to read off the sample.  The number of sample points above a quantile is close to Poisson
  // with mean lam, so "mean plus four standard deviations plus a constant" is almost never short.
  const double lam_lo = (double)p.k_target * (double)M / (double)p.d;
  const double lam_k = (double)p.k * (double)M / (double)p.d;
  const bool exact = (int64_t)M == p.d;
  const double r_lo_d = exact ? (double)p.k_target : ceil(lam_lo + 4.0 * sqrt(lam_lo) + 8.0);
  const double r_hi_d = exact ? (double)p.k : floor(lam_k - 4.0 * sqrt(lam_k) - 8.0);
  const u32 r_lo = r_lo_d > (double)M ? (u32)M + 1u : (u32)r_lo_d;
  const u32 r_hi = r_hi_d < 1.0 ? 1u : (u32)r_hi_d;

  // One suffix scan serves both ranks.  A thread owns 16 consecutive bins, counted from the top.
  constexpr int kPer = kSampleBins / kBlockSel;
  u32 mine[kPer];
  u32 sum = 0;
#pragma unroll
  for (int i = 0; i < kPer; ++i) {
    mine[i] = s_hist[sample_slot((u32)(kSampleBins - 1 - (tid * kPer + i)))];
    sum += mine[i];
  }
  __shared__ u32 s_frac[2];  // for the r_lo bin: sample points in it, and how many of them rank at or above r_lo
  if (tid == 0) { s_res[0] = kFull; s_res[1] = kFull; }
  u32 total;
  const u32 excl = block_excl_scan(sum, s_scan, &total);
  const u32 want[2] = {r_hi, r_lo};
#pragma unroll
  for (int w = 0; w < 2; ++w) {
    if (excl < want[w] && want[w] <= excl + sum) {
      u32 acc = excl;
#pragma unroll
      for (int i = 0; i < kPer; ++i) {
        if (acc < want[w] && want[w] <= acc + mine[i]) {
          s_res[w] = (u32)(kSampleBins - 1 - (tid * kPer + i));
          if (w == 1) { s_frac[0] = mine[i]; s_frac[1] = want[w] - acc; }
        }
        acc += mine[i];
      }
    }
  }
  __syncthreads();
  // upper end of the key range the select should resolve finely: the k-th largest score cannot
  // exceed the k-th largest |a|, estimated from above by the sample's r_hi-th largest
  u32 hi_key = s_res[0] == kFull ? 0x7F7FFFFFu : (((s_res[0] + 1u) << kSampleShift) - 1u);
  if (r_hi_d < 1.0) hi_key = hi_key < 0x7F000000u ? hi_key + (1u << 23) : 0x7F7FFFFFu;  // an octave of slack
  // the cutoff: inside the bin that holds the r_lo-th largest sample, placed as if the bin's sample
  // points were spread evenly over it (0: keep everything).  Error feedback piles entries up just
  // below the selection threshold, so a cutoff a whole bin too low would gather far too many.
  // Error feedback can pack a large part of a row into a band much narrower than a bin, right under the
  // selection threshold; that guess can then land above the whole band and leave fewer than k entries
  // above the cutoff (or below it and gather far too many).  The selection notices (it falls back to its dense
  // path, which is exact but slow) and asks for the next rounds' cutoffs to be resolved exactly: the sample's keys
  // are then read once more and the position inside the bin is found down to 32 key units (about 5 us more).
  u32 cutoff = 0u;
  if (r_lo <= (u32)M && s_res[1] != kFull) {
    const u32 width = 1u << kSampleShift;
    const u32 bin = s_res[1], in_bin = s_frac[0], need = s_frac[1];  // the same in every thread
    if (want_exact) {
      __syncthreads();  // every thread has read s_res / s_frac and its bins of s_hist
      for (int i = tid; i < kBins; i += blockDim.x) s_hist[i] = 0;
      __syncthreads();
      const u32* keys = p.skeys + (size_t)n * kSampleMax;
      const uint4* keys4 = reinterpret_cast<const uint4*>(keys);
      for (int i0 = 0; i0 < kSampleMax / 4; i0 += 8 * kBlockSel) {  // two rounds of eight 16-byte loads per thread
        uint4 kk[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) kk[q] = __ldcg(&keys4[i0 + q * kBlockSel + tid]);
#pragma unroll
        for (int q = 0; q < 8; ++q) {
          const u32 v[4] = {kk[q].x, kk[q].y, kk[q].z, kk[q].w};
#pragma unroll
          for (int z = 0; z < 4; ++z)
            if ((v[z] >> kSampleShift) == bin) atomicAdd(&s_hist[(v[z] >> (kSampleShift - 12)) & (u32)(kBins - 1)], 1u);
        }
      }
      __syncthreads();
      block_find_from_top(s_hist, kBins, need, s_scan, s_res);  // the sub-bin of the need-th largest key of the bin
      const u32 sub = s_res[0] == kFull ? 0u : s_res[0];
      cutoff = (bin << kSampleShift) + (sub << (kSampleShift - 12));
    } else {
      const u32 below = (u32)(((u64)(in_bin - need) * width) / (in_bin + 1u));  // offset from the bin's lower edge
      cutoff = (bin << kSampleShift) + below;
    }
  }
  if (tid == 0) {
    const u32 range = hi_key > cutoff ? hi_key - cutoff : 0u;
    u32 shift = 0;
    while ((range >> shift) > (u32)(kBins - 2)) ++shift;
    if (want_exact) ctl->exact_rounds -= 1u;
    ctl->hint = cutoff;
    // force_dense == 2: the dense path is asked for, on the whole grid; the cutoff only serves it as a hint
    ctl->cutoff = p.force_dense == 2 ? kFull : cutoff;
    ctl->bin_shift = shift;
    ctl->cand_count = 0;
    ctl->force_dense = p.force_dense == 2 ? 1u : 0u;
    ctl->bcount = 0;
    ctl->acount = 0;
    ctl->n_valid = 0;
    ctl->b1 = kFull; ctl->above1 = 0; ctl->go_dense = 0; ctl->took_dense = 0;
  }
}

// ---------------------------------------------------------------------------------------------
// k_stream: a = eps + g for all workers, in place; candidates appended.  Persistent grid, one
// warp per chunk of 512 or 1024 elements (see StreamShape), chunks dealt round-robin so that
// neighbouring warps read neighbouring memory.  12 (fp32) or 10 (bf16) bytes of HBM traffic per
// coordinate.
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
  const u32* marks;  // [N][W] last round's mask, or NULL: entries on it are not candidates (their
  int64_t W;         // regularised score comes from the override list instead)
  const u32* chunk_cut;  // layer-wise mode: [N][cuts] candidate cutoff per kCutSpan coordinates (the layers have
  int64_t cuts;          // their own thresholds), instead of one per worker; else NULL
};

// Write a warp's staged hits to the worker's candidate list.  With a previous mask, the entries on it
// are dropped first: the probes of a flush are issued four per lane at a time, so the warp waits for
// memory a few times per flush, not once per hit.
__device__ __forceinline__ void stream_flush(u64* list, u32& wcount, WorkerCtl* ctl, u64* cand,
                                             int64_t cap, const u32* marks, int lane) {
  __syncwarp();
  if (wcount) {
    if (marks) {
      u32 kept = 0;
      const u32 total = wcount;
#pragma unroll 1
      for (u32 r0 = 0; r0 < total; r0 += 128) {
        u64 ent[4];
        u32 word[4];
#pragma unroll
        for (int r = 0; r < 4; ++r) {
          const u32 i = r0 + (u32)r * 32 + lane;
          ent[r] = i < total ? list[i] : 0ull;
          word[r] = i < total ? __ldg(&marks[composite_idx(ent[r]) >> 5]) : 0u;
        }
        __syncwarp();  // every lane has read its entries before any is overwritten
#pragma unroll
        for (int r = 0; r < 4; ++r) {
          const u32 i = r0 + (u32)r * 32 + lane;
          const bool keep = i < total && !((word[r] >> (composite_idx(ent[r]) & 31)) & 1u);
          const u32 m = __ballot_sync(kFull, keep);
          if (keep) list[kept + __popc(m & ((1u << lane) - 1u))] = ent[r];  // kept <= r0 + 32 r: behind the reads
          kept += __popc(m);
        }
        __syncwarp();
      }
      wcount = kept;
    }
    if (wcount) {
      u32 base = 0;
      if (lane == 0) base = atomicAdd(&ctl->cand_count, wcount);
      base = __shfl_sync(kFull, base, 0);
      for (u32 i = lane; i < wcount; i += 32) {
        const u64 pos = (u64)base + i;
        if (pos < (u64)cap) cand[pos] = list[i];
      }
    }
  }
  wcount = 0;
  __syncwarp();
}

// Elements a lane handles per step, steps a warp keeps in flight, and resident blocks per SM.  What
// bounds this kernel is the number of bytes in flight per SM (loaded HBM latency is about 2 us) against
// the registers that costs.  Shapes chosen by measurement on a B200:
//   fp32: four elements per lane and step, eight steps (256 B per thread), two blocks per SM:
//         6.17 TB/s on 89 M coordinates (four steps and three blocks: 5.96-6.09; four blocks: 5.80);
//   bf16: eight elements per lane and step (one 16-byte gradient load), two steps (96 B per thread),
//         three blocks per SM: 6.11 TB/s on 996 M coordinates (four steps, two blocks: 4.98-5.27;
//         8-byte gradient loads: 3.8).
#ifndef REGTOPK_STREAM_STEPS_F32
#define REGTOPK_STREAM_STEPS_F32 8
#endif
#ifndef REGTOPK_STREAM_STEPS_BF16
#define REGTOPK_STREAM_STEPS_BF16 2
#endif
#ifndef REGTOPK_STREAM_EPL_BF16
#define REGTOPK_STREAM_EPL_BF16 8
#endif
#ifndef REGTOPK_STREAM_BLOCKS_INPLACE
#define REGTOPK_STREAM_BLOCKS_INPLACE 3
#endif
template <bool BF16, bool VEC, bool INPLACE = false>
struct StreamShape {
  static constexpr int kEpl = (BF16 && VEC) ? REGTOPK_STREAM_EPL_BF16 : 4;  // elements per lane and step
  static constexpr int kVec = kEpl / 4;                     // float4 vectors per lane and step
  static constexpr int kStep = 32 * kEpl;                   // elements per warp and step
  static constexpr int kSteps = (BF16 && VEC) ? REGTOPK_STREAM_STEPS_BF16 : (VEC ? REGTOPK_STREAM_STEPS_F32 : 4);
  static constexpr int kChunk = kStep * kSteps;             // elements per warp iteration (divides 1024)
#ifndef REGTOPK_STREAM_BLOCKS_F32
#define REGTOPK_STREAM_BLOCKS_F32 2
#endif
#ifndef REGTOPK_STREAM_BLOCKS_BF16
#define REGTOPK_STREAM_BLOCKS_BF16 3
#endif
  static constexpr int kBlocksPerSm = INPLACE ? REGTOPK_STREAM_BLOCKS_INPLACE
                                      : (BF16 && VEC) ? REGTOPK_STREAM_BLOCKS_BF16 : (VEC ? REGTOPK_STREAM_BLOCKS_F32 : 2);
};

// INPLACE: the rows of eps already hold a = eps + g (the caller added its gradients there); nothing but
// those rows is read and nothing is written back: 4 bytes of HBM traffic per coordinate.
template <bool BF16, bool VEC, bool INPLACE>
__global__ void __launch_bounds__(kStreamThreads, StreamShape<BF16, VEC, INPLACE>::kBlocksPerSm) k_stream(StreamArgs p) {
  typedef StreamShape<BF16, VEC, INPLACE> S;
  __shared__ u64 s_list[kStreamThreads / 32][kWarpList];
  grid_dependency_begin();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  u64* list = s_list[warp];
  u32 wcount = 0;  // warp-uniform
  const int64_t chunks_per_row = (p.d + S::kChunk - 1) / S::kChunk;
  const int64_t total = chunks_per_row * p.N;
  const int64_t nwarps = (int64_t)gridDim.x * (kStreamThreads / 32);
  int cur_n = -1;
  u32 cutoff = kFull;
  float* eps_row = nullptr;
  const char* grow = nullptr;
  const u32* marks = nullptr;

  // row and position of the warp's chunk advance incrementally: one 64-bit division up front, none per chunk
  const int64_t cfirst = (int64_t)blockIdx.x * (kStreamThreads / 32) + warp;
  int64_t row = cfirst / chunks_per_row, in_row = cfirst - row * chunks_per_row;
  const int64_t step_rows = nwarps / chunks_per_row, step_in = nwarps - step_rows * chunks_per_row;
  for (int64_t c = cfirst; c < total; c += nwarps) {
    const int n = (int)row;
    const int64_t base = in_row * S::kChunk;
    row += step_rows;
    in_row += step_in;
    if (in_row >= chunks_per_row) { in_row -= chunks_per_row; ++row; }
    if (n != cur_n) {
      if (cur_n >= 0) stream_flush(list, wcount, p.ctl + cur_n, p.cand + (size_t)cur_n * p.stride, p.cap, marks, lane);
      cur_n = n;
      cutoff = p.ctl[n].cutoff;
      eps_row = p.eps + (size_t)n * p.ld;
      grow = static_cast<const char*>(p.grads) + (size_t)n * p.grad_ld * (BF16 ? 2 : 4);
      marks = p.marks ? p.marks + (size_t)n * p.W : nullptr;
    }
    const bool full = base + S::kChunk <= p.d;  // warp-uniform
    if (p.chunk_cut) {  // layer-wise: the lowest cutoff of the layers this chunk meets (admits a superset)
      const u32* cc = p.chunk_cut + (size_t)n * p.cuts + base / kCutSpan;
      cutoff = __ldg(cc);
#pragma unroll
      for (int i = 1; i < S::kChunk / kCutSpan; ++i)
        if (base + (int64_t)i * kCutSpan < p.d) cutoff = min(cutoff, __ldg(cc + i));
    }
    float4 e[S::kSteps][S::kVec], g[S::kSteps][S::kVec];
#pragma unroll
    for (int u = 0; u < S::kSteps; ++u) {
      const int64_t j = base + u * S::kStep + lane * S::kEpl;
#pragma unroll
      for (int v = 0; v < S::kVec; ++v)
        e[u][v] = __ldcs(reinterpret_cast<const float4*>(eps_row + j + 4 * v));  // rows are padded: in bounds
      if (INPLACE) {
        // no gradient to load
      } else if (VEC && (full || j + S::kEpl - 1 < p.d)) {
        if (BF16) {
          if (S::kEpl == 8) {  // eight bf16 in one 16-byte load
            const uint4 raw = __ldcs(reinterpret_cast<const uint4*>(grow + j * 2));
            g[u][0].x = __uint_as_float(raw.x << 16);
            g[u][0].y = __uint_as_float(raw.x & 0xFFFF0000u);
            g[u][0].z = __uint_as_float(raw.y << 16);
            g[u][0].w = __uint_as_float(raw.y & 0xFFFF0000u);
            g[u][S::kVec - 1].x = __uint_as_float(raw.z << 16);
            g[u][S::kVec - 1].y = __uint_as_float(raw.z & 0xFFFF0000u);
            g[u][S::kVec - 1].z = __uint_as_float(raw.w << 16);
            g[u][S::kVec - 1].w = __uint_as_float(raw.w & 0xFFFF0000u);
          } else {  // four bf16 in one 8-byte load
            const uint2 raw = __ldcs(reinterpret_cast<const uint2*>(grow + j * 2));
            g[u][0].x = __uint_as_float(raw.x << 16);
            g[u][0].y = __uint_as_float(raw.x & 0xFFFF0000u);
            g[u][0].z = __uint_as_float(raw.y << 16);
            g[u][0].w = __uint_as_float(raw.y & 0xFFFF0000u);
          }
        } else {
          g[u][0] = __ldcs(reinterpret_cast<const float4*>(grow + j * 4));
        }
      } else {
#pragma unroll
        for (int v = 0; v < S::kVec; ++v) {
          const int64_t jj = j + 4 * v;
          g[u][v].x = (jj + 0 < p.d) ? load_grad<BF16>(grow, jj + 0) : 0.0f;
          g[u][v].y = (jj + 1 < p.d) ? load_grad<BF16>(grow, jj + 1) : 0.0f;
          g[u][v].z = (jj + 2 < p.d) ? load_grad<BF16>(grow, jj + 2) : 0.0f;
          g[u][v].w = (jj + 3 < p.d) ? load_grad<BF16>(grow, jj + 3) : 0.0f;
        }
      }
    }
#pragma unroll
    for (int u = 0; u < S::kSteps; ++u) {
#pragma unroll
      for (int v = 0; v < S::kVec; ++v) {
        const int64_t j = base + u * S::kStep + lane * S::kEpl + 4 * v;
        float4 a;
        if (INPLACE) {
          a = e[u][v];
        } else {
          a.x = __fadd_rn(e[u][v].x, g[u][v].x);
          a.y = __fadd_rn(e[u][v].y, g[u][v].y);
          a.z = __fadd_rn(e[u][v].z, g[u][v].z);
          a.w = __fadd_rn(e[u][v].w, g[u][v].w);
          __stcs(reinterpret_cast<float4*>(eps_row + j), a);  // padding receives 0 + 0; streaming store: the
                                                              // accumulators should not push the small lists out of L2
        }
#if !REGTOPK_DEBUG
        if (full) {
          // Inside the row one compare decides for the quad: the largest key is the key of the largest magnitude
          // (three maxima with free |.| operands instead of four masks and four compares; the read-only variant
          // of this kernel is bound by instruction issue, not by memory).
          const float top = fmaxf(fmaxf(fabsf(a.x), fabsf(a.y)), fmaxf(fabsf(a.z), fabsf(a.w)));
          if (!__any_sync(kFull, __float_as_uint(top) >= cutoff)) continue;
        }
#endif
        const u32 k0 = __float_as_uint(a.x) & 0x7FFFFFFFu, k1 = __float_as_uint(a.y) & 0x7FFFFFFFu;
        const u32 k2 = __float_as_uint(a.z) & 0x7FFFFFFFu, k3 = __float_as_uint(a.w) & 0x7FFFFFFFu;
        RT_NOTE_NONFINITE(k0, full || j + 0 < p.d); RT_NOTE_NONFINITE(k1, full || j + 1 < p.d);
        RT_NOTE_NONFINITE(k2, full || j + 2 < p.d); RT_NOTE_NONFINITE(k3, full || j + 3 < p.d);
        const bool h0 = k0 >= cutoff && (full || j + 0 < p.d);
        const bool h1 = k1 >= cutoff && (full || j + 1 < p.d);
        const bool h2 = k2 >= cutoff && (full || j + 2 < p.d);
        const bool h3 = k3 >= cutoff && (full || j + 3 < p.d);
        if (__any_sync(kFull, h0 | h1 | h2 | h3)) {
          const u32 lt = (1u << lane) - 1u;
          u32 m;
          m = __ballot_sync(kFull, h0);
          if (h0 && RT_INB(wcount + __popc(m & lt) < (u32)kWarpList)) list[wcount + __popc(m & lt)] = make_composite(k0, (u32)j);
          wcount += __popc(m);
          m = __ballot_sync(kFull, h1);
          if (h1 && RT_INB(wcount + __popc(m & lt) < (u32)kWarpList)) list[wcount + __popc(m & lt)] = make_composite(k1, (u32)j + 1);
          wcount += __popc(m);
          m = __ballot_sync(kFull, h2);
          if (h2 && RT_INB(wcount + __popc(m & lt) < (u32)kWarpList)) list[wcount + __popc(m & lt)] = make_composite(k2, (u32)j + 2);
          wcount += __popc(m);
          m = __ballot_sync(kFull, h3);
          if (h3 && RT_INB(wcount + __popc(m & lt) < (u32)kWarpList)) list[wcount + __popc(m & lt)] = make_composite(k3, (u32)j + 3);
          wcount += __popc(m);
          if (wcount >= kWarpList - 128)  // the next four elements per lane add at most 128
            stream_flush(list, wcount, p.ctl + cur_n, p.cand + (size_t)cur_n * p.stride, p.cap, marks, lane);
        }
      }
    }
  }
  if (cur_n >= 0) stream_flush(list, wcount, p.ctl + cur_n, p.cand + (size_t)cur_n * p.stride, p.cap, marks, lane);
}

// ---------------------------------------------------------------------------------------------
// k_post: one thread-block cluster per worker.  The cluster's blocks meet only at the hardware
// cluster barrier; what they exchange (histograms, list lengths, segment totals) goes through
// global memory, which the barrier's release/acquire makes visible.  Every block of a cluster
// reaches every barrier: all branches that contain one depend only on values that are the same in
// all blocks of the cluster.
// ---------------------------------------------------------------------------------------------
struct PostShared {
  u32 hist[kBins];    // histogram of this block, then of the cluster
  u32 spare[kBins];   // with hist: 8192 words reused as item storage and per-warp emission lists
  u32 fres[3];
  u32 scan[33];
  u32 cnt;
};

struct PostArgs {
  WorkerCtl* ctl;
  GlobalCtl* gctl;
  float* eps;  // holds a after k_stream; winners are zeroed here
  int64_t ld;
  int64_t d;
  int64_t k;
  const float* g_prev;
  const int32_t* prev_idx;
  const float* prev_val;
  const float* omega;
  float mu;
  u32* ovr_key;   // [N][k] score bits of every previous-support entry
  u64* ovr_comp;  // [N][k] composite if the score reaches the cutoff, else 0
  u64* candA;     // [N][stride]; k_stream filled at most capA entries of a row
  u64* candB;     // [N][stride]
  int64_t capA;
  int64_t stride;  // capA + k: what one histogram bin can hold (all candidates plus all overrides)
  u32* ghist;      // [N][4][kBins] cluster-wide histograms, zeroed by k_sample_cutoff
  u32* shist;      // [N][kSampleBins] histogram of k_sample_cutoff, cleared here for the next round
  u32* btot;       // [N][2][kMaxCluster] per-block totals
  const u32* mask_old;  // [N][W] last round's mask (marks the previous support)
  u32* mask_new;   // [N][W] this round's mask; on entry it holds the mask of two rounds ago
  u32* qprefix;    // [N][W/4] mask bits before each quad (4 words) within its segment
  u32* segtot;     // [N][kMaxSegments] mask bits of each segment
  u32* segbase;    // [N][kMaxSegments] mask bits before each segment (written for k_aggregate)
  int64_t W;       // words per row, a multiple of 32
  int32_t* out_idx;
  float* out_val;
  int32_t* cur_idx;  // on entry: the pairs of two rounds ago (the bits to clear in mask_new)
  float* cur_val;
  int use_marks;  // previous support carries regularised scores (round >= 1, mu > 0)
  int has_stale;  // mask_new holds an old mask (round >= 2)
  int pair_mode;  // many pairs: emit (index, value) as one store into the B list; k_unzip follows
  int wide;       // k_post runs between the wide kernels: refinement or dense path only
  int grid_dense; // a worker that needs the dense exact path is left to k_dense (ctl->go_dense) instead of this cluster
};

__device__ __forceinline__ u32 warp_reserve_global(bool pred, u32* counter) {
  const u32 m = __ballot_sync(kFull, pred);
  if (m == 0) return 0;
  const int lane = threadIdx.x & 31;
  const int leader = __ffs(m) - 1;
  u32 base = 0;
  if (lane == leader) base = atomicAdd(counter, (u32)__popc(m));
  base = __shfl_sync(kFull, base, leader);
  return base + (u32)__popc(m & ((1u << lane) - 1u));
}

__device__ __forceinline__ void set_winner(u32* mask, u32 idx, int64_t d) {
  if (RT_INB((int64_t)idx < d)) atomicOr(&mask[idx >> 5], 1u << (idx & 31));
}

__device__ __forceinline__ u32 select_bin(u32 key, u32 cutoff, u32 shift) {
  const u32 b = (key - cutoff) >> shift;
  return b < (u32)(kBins - 1) ? b : (u32)(kBins - 1);
}

// After the cluster barrier: every block loads the cluster's histogram and finds the bin of the
// r-th entry from the top by itself (all blocks get the same answer).
__device__ __forceinline__ void load_and_find(PostShared& sh, const u32* g_hist, u32 r, u32* bin,
                                              u32* above, u32* total) {
  for (int i = threadIdx.x; i < kBins; i += blockDim.x) sh.hist[i] = __ldcg(&g_hist[i]);
  __syncthreads();
  block_find_from_top(sh.hist, kBins, r, sh.scan, sh.fres);
  *bin = sh.fres[0];
  *above = sh.fres[1];
  *total = sh.fres[2];
  __syncthreads();
}

// Score key of entry j for the dense path: the override's on the previous support, bits(|a|) elsewhere.
__device__ __forceinline__ u32 dense_key(const PostArgs& p, int n, int64_t j) {
  if (p.use_marks) {
    const u32 w = p.mask_old[(size_t)n * p.W + (j >> 5)];
    if ((w >> (j & 31)) & 1u) {
      const int32_t* pi = p.prev_idx + (size_t)n * p.k;
      int64_t lo = 0, hi = p.k;
      while (lo < hi) {
        const int64_t mid = (lo + hi) >> 1;
        if (pi[mid] < (int32_t)j) lo = mid + 1; else hi = mid;
      }
      return __ldcg(&p.ovr_key[(size_t)n * p.k + lo]);
    }
  }
  return __float_as_uint(p.eps[(size_t)n * p.ld + j]) & 0x7FFFFFFFu;
}

// The same for the four entries j4 .. j4 + 3 (j4 a multiple of 4; rows are 16-byte aligned and padded): one
// 16-byte load of the residuals and one mask word; only entries on the previous support, which are few, take the
// search.  Keys of entries at or beyond `end` are 0 and not to be used.
__device__ __forceinline__ void dense_keys4(const PostArgs& p, int n, int64_t j4, int64_t end, u32 (&key)[4]) {
  key[0] = key[1] = key[2] = key[3] = 0u;
  if (j4 >= end) return;
  const float4 e = *reinterpret_cast<const float4*>(p.eps + (size_t)n * p.ld + j4);
  const u32 w = p.use_marks ? (p.mask_old[(size_t)n * p.W + (j4 >> 5)] >> (j4 & 31)) & 15u : 0u;
  const float v[4] = {e.x, e.y, e.z, e.w};
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    if (j4 + q >= end) break;
    key[q] = ((w >> q) & 1u) ? dense_key(p, n, j4 + q) : (__float_as_uint(v[q]) & 0x7FFFFFFFu);
  }
}

// One block: among list[0..count) (count <= blockDim.x, unique composites) set the `need` largest as
// winners, but only those whose mask word lies in [w0, w1) (the caller's share of the mask).
__device__ void refine_small(PostShared& sh, u32* mask, int64_t d, const u64* list, u32 count, u32 need,
                             int64_t w0, int64_t w1) {
  u64* s_items = reinterpret_cast<u64*>(sh.hist);
  const int tid = threadIdx.x;
  u64 mine = 0ull;
  if ((u32)tid < count) {
    mine = __ldcg(&list[tid]);
    s_items[tid] = mine;
  }
  __syncthreads();
  if ((u32)tid < count) {
    const u32 idx = composite_idx(mine);
    const int64_t wi = (int64_t)(idx >> 5);
    if (wi >= w0 && wi < w1) {
      u32 above = 0;
      for (u32 j = 0; j < count; ++j) above += s_items[j] > mine ? 1u : 0u;
      if (above < need) set_winner(mask, idx, d);
    }
  }
  __syncthreads();
}

// Leader block only: the `need` largest composites of list[0..count), any count (long runs of equal
// keys end up here).  Eight histogram passes over the list fix the need-th largest composite byte by
// byte, without moving the list; a last pass sets everything at or above it.
__device__ void refine_large(PostShared& sh, u32* mask, int64_t d, GlobalCtl* gctl, const u64* list, u32 count,
                             u32 need) {
  const int tid = threadIdx.x;
  if (need == 0) return;
  u64 prefix = 0ull;  // the bytes of the need-th largest composite fixed so far
  for (int shift = 56; shift >= 0; shift -= 8) {
    for (int i = tid; i < 256; i += blockDim.x) sh.hist[i] = 0;
    __syncthreads();
    for (u32 i = tid; i < count; i += blockDim.x) {
      const u64 c = __ldcg(&list[i]);
      if (shift == 56 || (c >> (shift + 8)) == prefix) atomicAdd(&sh.hist[(u32)(c >> shift) & 255u], 1u);
    }
    __syncthreads();
    block_find_from_top(sh.hist, 256, need, sh.scan, sh.fres);
    const u32 b = sh.fres[0], above = sh.fres[1];
    __syncthreads();
    if (b == kFull) {  // cannot happen while need <= count
      if (tid == 0) atomicOr(&gctl->err, kErrRefine);
      return;
    }
    need -= above;
    prefix = (prefix << 8) | (u64)b;
  }
  for (u32 i = tid; i < count; i += blockDim.x) {
    const u64 c = __ldcg(&list[i]);
    if (c >= prefix) set_winner(mask, composite_idx(c), d);
  }
}

__device__ __forceinline__ u32 popc4(const uint4& v) {
  return (u32)(__popc(v.x) + __popc(v.y) + __popc(v.z) + __popc(v.w));
}

// ---- pieces of the selection, shared by k_post (one cluster per worker) and the wide kernels (the whole
//      grid split over the workers; used when N*k is large).  first_t / stride_t: this thread's index
//      among, and the number of, the threads that work on worker n's row. ----

// One sweep over the lists, a single wave of coalesced loads per step:
//   (a) the mask buffer of this round still holds the mask of two rounds ago: clear those words;
//   (b) the override scores (written by k_sample_cutoff's override clusters) that reach the cutoff
//       become composites and enter the histogram;
//   (c) the candidates (k_stream already dropped those on the previous support) enter it too.
__device__ __forceinline__ void post_sweep(const PostArgs& p, int n, u32 first_t, u32 stride_t, bool dense,
                                           u32 ncand, u32 cutoff, u32 bshift, u32* s_hist) {
  const u32 k = (u32)p.k;
  const size_t obase = (size_t)n * p.k;
  const u64* A = p.candA + (size_t)n * p.stride;
  u64* O = p.ovr_comp + obase;
  const u32* okey = p.ovr_key + obase;
  const int32_t* prev_idx = p.prev_idx + obase;
  u32* mask = p.mask_new + (size_t)n * p.W;
  const u32 span = !dense && ncand > k ? ncand : k;
  constexpr int kP0 = 8;  // items per thread in flight
  for (u32 i0 = first_t; i0 < span; i0 += kP0 * stride_t) {
    int32_t stale[kP0], j[kP0];
    u32 key[kP0];
    u64 c[kP0];
#pragma unroll
    for (int q = 0; q < kP0; ++q) {
      const u32 i = i0 + q * stride_t;
      const bool in_k = i < k;
      stale[q] = (in_k && p.has_stale) ? p.cur_idx[obase + i] : -1;
      j[q] = (in_k && p.use_marks) ? prev_idx[i] : -1;
      key[q] = (in_k && p.use_marks) ? okey[i] : 0u;
      c[q] = (!dense && i < ncand) ? A[i] : 0ull;
    }
#pragma unroll
    for (int q = 0; q < kP0; ++q) {
      const u32 i = i0 + q * stride_t;
      if (stale[q] >= 0 && RT_INB((int64_t)stale[q] < p.d)) mask[(u32)stale[q] >> 5] = 0u;
      if (j[q] >= 0) {
        const u64 oc = key[q] >= cutoff ? make_composite(key[q], (u32)j[q]) : 0ull;
        O[i] = oc;
        if (!dense && oc) atomicAdd(&s_hist[select_bin(key[q], cutoff, bshift)], 1u);
      }
      if (c[q]) atomicAdd(&s_hist[select_bin((u32)(c[q] >> 32), cutoff, bshift)], 1u);
    }
  }
}

// Classify candidates and overrides (one item list, eight loads per thread in flight): above the threshold
// bin -> winner; inside it -> refinement list.  Whole warps must call it.
__device__ __forceinline__ void post_classify(const PostArgs& p, int n, u32 first_t, u32 stride_t, u32 ncand,
                                              u32 novr, u32 cutoff, u32 bshift, u32 b1) {
  const u64* A = p.candA + (size_t)n * p.stride;
  u64* B = p.candB + (size_t)n * p.stride;
  const u64* O = p.ovr_comp + (size_t)n * p.k;
  u32* mask = p.mask_new + (size_t)n * p.W;
  WorkerCtl* ctl = p.ctl + n;
  const u32 total_items = ncand + novr;
  const u32 iters = (total_items + 8 * stride_t - 1) / (8 * stride_t);
  for (u32 it = 0; it < iters; ++it) {
    u64 c[8];
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      const u32 t = (it * 8 + q) * stride_t + first_t;
      c[q] = t < ncand ? __ldcg(A + t) : (t < total_items ? __ldcg(O + (t - ncand)) : 0ull);
    }
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      const u32 bin = c[q] ? select_bin((u32)(c[q] >> 32), cutoff, bshift) : 0u;
      if (c[q] && bin > b1) set_winner(mask, composite_idx(c[q]), p.d);
      const bool inbin = c[q] && bin == b1;
      const u32 pos = warp_reserve_global(inbin, &ctl->bcount);
      if (inbin && RT_INB((int64_t)pos < p.stride)) B[pos] = c[q];
    }
  }
}

// One warp: per quad (four mask words, 128 coordinates) of segment `seg`, the mask bits before it inside
// the segment; the segment's total.  Segments are runs of seg_units 8-word units of the mask row.
__device__ __forceinline__ void post_prefix_segment(const PostArgs& p, int n, u32 seg, int64_t seg_units, int lane) {
  const int64_t U = p.W >> 3;
  const uint4* quads = reinterpret_cast<const uint4*>(p.mask_new + (size_t)n * p.W);
  u32* qpre = p.qprefix + (size_t)n * (p.W >> 2);
  const int64_t wu0 = (int64_t)seg * seg_units < U ? (int64_t)seg * seg_units : U;
  const int64_t wu1 = wu0 + seg_units < U ? wu0 + seg_units : U;
  u32 running = 0;
  for (int64_t ub = wu0; ub < wu1; ub += 128) {  // four rows of 32 units per step
    uint4 x[4], y[4];
#pragma unroll
    for (int it = 0; it < 4; ++it) {
      const int64_t u = ub + it * 32 + lane;
      x[it] = u < wu1 ? __ldcg(quads + 2 * u) : make_uint4(0, 0, 0, 0);
      y[it] = u < wu1 ? __ldcg(quads + 2 * u + 1) : make_uint4(0, 0, 0, 0);
    }
#pragma unroll
    for (int it = 0; it < 4; ++it) {
      const u32 cx = popc4(x[it]), c = cx + popc4(y[it]);
      u32 inc = c;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const u32 t = __shfl_up_sync(kFull, inc, o);
        if (lane >= o) inc += t;
      }
      const int64_t u = ub + it * 32 + lane;
      const u32 pre = running + inc - c;
      if (u < wu1) *reinterpret_cast<uint2*>(qpre + 2 * u) = make_uint2(pre, pre + cx);
      running += __shfl_sync(kFull, inc, 31);
    }
  }
  if (lane == 0) p.segtot[(size_t)n * kMaxSegments + seg] = running;
}

// Every item whose mask bit is set looks its rank up (segment base + quad prefix + bits before it in
// the quad), writes its (index, value) pair there and zeroes its residual.  Normal path: candidates and
// overrides as one item list; dense path: its k winners, nothing else.  Items below the threshold bin
// cannot have won and are skipped without touching memory.
__device__ __forceinline__ void post_emit(const PostArgs& p, int n, u32 first_t, u32 stride_t, u32 ncand, u32 novr,
                                          bool took_dense, u32 cutoff, u32 bshift, u32 b1, const u32* s_segbase,
                                          int64_t seg_units) {
  const u32 k = (u32)p.k;
  const size_t obase = (size_t)n * p.k;
  const u64* A = p.candA + (size_t)n * p.stride;
  u64* B = p.candB + (size_t)n * p.stride;
  const u64* O = p.ovr_comp + obase;
  float* eps_row = p.eps + (size_t)n * p.ld;
  const uint4* quads = reinterpret_cast<const uint4*>(p.mask_new + (size_t)n * p.W);
  const u32* qpre = p.qprefix + (size_t)n * (p.W >> 2);
  const u32 nA = took_dense ? k : ncand;
  const u32 total_items = nA + (took_dense ? 0u : novr);
  if (took_dense) A = O;  // every flavour of the dense path leaves its k winners in the override-composite row
  for (u32 t0 = first_t; t0 < total_items; t0 += 4 * stride_t) {
    u64 c[4];
    uint4 qw[4];
    u32 qp[4];
    float vv[4];
    bool live[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const u32 t = t0 + q * stride_t;
      c[q] = t < nA ? __ldcg(A + t) : (t < total_items ? __ldcg(O + (t - nA)) : 0ull);
    }
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const u32 idx = composite_idx(c[q]);
      live[q] = c[q] != 0ull && (took_dense || select_bin((u32)(c[q] >> 32), cutoff, bshift) >= b1) && RT_INB((int64_t)idx < p.d);
      qw[q] = live[q] ? __ldcg(quads + (idx >> 7)) : make_uint4(0, 0, 0, 0);
      qp[q] = live[q] ? __ldcg(qpre + (idx >> 7)) : 0u;
      vv[q] = live[q] ? eps_row[idx] : 0.0f;
    }
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      if (!live[q]) continue;
      const u32 idx = composite_idx(c[q]);
      const u32 w[4] = {qw[q].x, qw[q].y, qw[q].z, qw[q].w};
      const u32 wsel = (idx >> 5) & 3u;
      u32 before = 0, word = 0;
#pragma unroll
      for (int wi = 0; wi < 4; ++wi) {
        if ((u32)wi < wsel) before += __popc(w[wi]);
        if ((u32)wi == wsel) word = w[wi];
      }
      const u32 bm = 1u << (idx & 31);
      if ((word & bm) && RT_INB((idx >> 8) / (u32)seg_units < (u32)kMaxSegments)) {
        const u32 r = s_segbase[(idx >> 8) / (u32)seg_units] + qp[q] + before + __popc(word & (bm - 1u));
        if (!RT_INB(r < k)) continue;
        eps_row[idx] = 0.0f;  // a - a
        if (p.pair_mode) {
          // many pairs: one 8-byte store at the (random) rank instead of four 4-byte ones; k_unzip
          // spreads the pairs over the four output arrays with sequential accesses afterwards
          reinterpret_cast<uint2*>(B)[r] = make_uint2(idx, __float_as_uint(vv[q]));
        } else {
          p.out_idx[obase + r] = (int32_t)idx;
          p.out_val[obase + r] = vv[q];
          p.cur_idx[obase + r] = (int32_t)idx;
          p.cur_val[obase + r] = vv[q];
        }
      }
    }
  }
}

__global__ void __launch_bounds__(kBlockPost, 1024 / kBlockPost) k_post(PostArgs p) {
  __shared__ __align__(16) PostShared sh;
  grid_dependency_begin();
  cg::cluster_group cl = cg::this_cluster();
  const u32 CS = cl.num_blocks(), rk = cl.block_rank();
  const int n = blockIdx.x / CS;
  const int tid = threadIdx.x;
  const u32 stride_t = CS * blockDim.x;        // threads of the cluster
  const u32 first_t = rk * blockDim.x + tid;   // this thread's index among them
  WorkerCtl* ctl = p.ctl + n;
  const u32 cutoff = ctl->cutoff, bshift = ctl->bin_shift;
  const u32 cand_count = ctl->cand_count;
  bool dense = ctl->force_dense != 0;          // the same in every block: nothing writes it here
  const u32 k = (u32)p.k;
  u64* A = p.candA + (size_t)n * p.stride;
  u64* B = p.candB + (size_t)n * p.stride;
  u32* mask = p.mask_new + (size_t)n * p.W;
  u32* ghist = p.ghist + (size_t)n * 4 * kBins;
  u32* btot = p.btot + (size_t)n * 2 * kMaxCluster;
  const bool overflow = (u64)cand_count > (u64)p.capA;
  const u32 ncand = overflow ? (u32)p.capA : cand_count;
  const u32 novr = p.use_marks ? k : 0u;
  // The mask row is cut into one segment of 8-word units per warp of the cluster; a block's share
  // is the segments of its warps.  The refinement and the emission both use this partition, so a
  // block only ever reads mask words whose last writers it has met at a barrier.
  const int64_t U = p.W >> 3;
  const int nw = blockDim.x >> 5;
  const u32 nseg = CS * (u32)nw;
  const int64_t seg_units = (U + nseg - 1) / nseg;
  const int64_t su0 = (int64_t)rk * nw * seg_units < U ? (int64_t)rk * nw * seg_units : U;
  const int64_t su1 = (int64_t)(rk + 1) * nw * seg_units < U ? (int64_t)(rk + 1) * nw * seg_units : U;

  u32 b1 = kFull, above1 = 0, nvalid = 0;
  bool took_dense = false;
  if (p.wide) {
    // the sweep, the threshold and the classification were done by k_wide_hist and k_wide_classify
    b1 = ctl->b1;
    above1 = ctl->above1;
    dense = ctl->go_dense != 0;
  } else {
    for (int i = tid; i < kBins; i += blockDim.x) sh.hist[i] = 0;
    for (u32 i = first_t; i < (u32)kSampleBins; i += stride_t) p.shist[(size_t)n * kSampleBins + i] = 0;
    __syncthreads();
    post_sweep(p, n, first_t, stride_t, dense, ncand, cutoff, bshift, sh.hist);
    __syncthreads();
    if (!dense) flush_hist(sh.hist, ghist, kBins);
    cl.sync();  // (1) cluster histogram complete; stale mask words cleared; override keys written
    if (!dense) {
      load_and_find(sh, ghist, k, &b1, &above1, &nvalid);
      if (b1 == kFull || overflow) dense = true;  // cutoff guessed too high, or the list overflowed
      if (rk == 0 && tid == 0) {
        ctl->n_valid = nvalid;
        if (dense) ask_for_exact_cutoffs(&ctl->exact_rounds, &ctl->exact_window);
      }
    }
    if (!dense) {
      post_classify(p, n, first_t, stride_t, ncand, novr, cutoff, bshift, b1);
      cl.sync();  // (2) refinement list complete
    }
  }
  if (dense && p.grid_dense) {  // the same in every block: k_dense, the next kernel, selects for this worker
    if (rk == 0 && tid == 0) {
      ctl->go_dense = 1u;
      atomicAdd(&p.gctl->dense_workers, 1ull);
    }
    return;
  }

  if (!dense) {
    const u32 nB = __ldcg(&ctl->bcount);
    const u32 need = k - above1;
    if (nB <= blockDim.x) {
      // every block ranks the short list itself and sets the winners of its own share of the mask
      refine_small(sh, mask, p.d, B, nB, need, su0 * 8, su1 * 8);
    } else if (nB <= k) {
      // A crowded threshold bin (error feedback packs the entries under the threshold into a band that a few
      // bins cover): a second histogram over that bin's own key range, 4096 sub-bins, by the whole cluster;
      // what is left in the sub-bin of the threshold (keys equal or nearly so) goes to the list refinement.
      // The second list lives behind the candidates in A (k entries are free there).
      const u32 lo2 = cutoff + (b1 << bshift);  // lower edge of the threshold bin; every listed key is at or above it
      u32 shift2 = bshift > 12u ? bshift - 12u : 0u;
      if (b1 == (u32)(kBins - 1)) {  // the clamped top bin reaches up to the largest key
        shift2 = 0;
        while (((0x7FFFFFFFu - lo2) >> shift2) > (u32)(kBins - 2)) ++shift2;
      }
      u64* B2 = A + p.capA;
      __syncthreads();
      for (int i = tid; i < kBins; i += blockDim.x) sh.hist[i] = 0;
      __syncthreads();
      for (u32 i = first_t; i < nB; i += stride_t)
        atomicAdd(&sh.hist[select_bin((u32)(__ldcg(B + i) >> 32), lo2, shift2)], 1u);
      __syncthreads();
      flush_hist(sh.hist, ghist + kBins, kBins);  // the second of the four histograms: unused on this path so far
      cl.sync();  // (2c) histogram of the threshold bin complete
      u32 b2, above2, total2;
      load_and_find(sh, ghist + kBins, need, &b2, &above2, &total2);  // need <= nB: always found
      const u32 iters2 = (nB + stride_t - 1) / stride_t;
      for (u32 it = 0; it < iters2; ++it) {
        const u32 i = it * stride_t + first_t;
        const u64 c = i < nB ? __ldcg(B + i) : 0ull;
        const u32 sub = c ? select_bin((u32)(c >> 32), lo2, shift2) : 0u;
        if (c && b2 != kFull && sub > b2) set_winner(mask, composite_idx(c), p.d);
        const bool inb = c && sub == b2;
        const u32 pos = warp_reserve_global(inb, &ctl->acount);  // acount: otherwise the dense path's counter
        if (inb && RT_INB(pos < k)) B2[pos] = c;
      }
      cl.sync();  // (2d) second list complete
      const u32 nB2 = __ldcg(&ctl->acount);
      const u32 need2 = need - above2;
      if (b2 == kFull) {
        if (rk == 0 && tid == 0) atomicOr(&p.gctl->err, kErrRefine);  // cannot happen while need <= nB
      } else if (nB2 <= blockDim.x) {
        refine_small(sh, mask, p.d, B2, nB2, need2, su0 * 8, su1 * 8);
      } else {
        if (rk == 0) refine_large(sh, mask, p.d, p.gctl, B2, nB2, need2);
        cl.sync();  // (2e) the leader's winners are set
      }
    } else {
      if (rk == 0) refine_large(sh, mask, p.d, p.gctl, B, nB, need);
      cl.sync();  // (2b) the leader's winners are set
    }
  } else {
    // ---- exact selection over the whole row: three radix digits of the 31-bit key ----
    took_dense = true;
    u64* Wl = p.ovr_comp + (size_t)n * p.k;  // the winners' list (the row is free on this path: see post_emit)
    if (rk == 0 && tid == 0) atomicAdd(&p.gctl->dense_workers, 1ull);
    // this block's part of the row; the cuts are multiples of four so that every thread reads whole quads
    const int64_t c0 = (int64_t)(((u64)rk * (u64)p.d) / CS) & ~(int64_t)3;
    const int64_t c1 = rk + 1 == CS ? p.d : (int64_t)(((u64)(rk + 1) * (u64)p.d) / CS) & ~(int64_t)3;
    u32 need = k, prefix = 0;
    bool bad = false;
    const int shifts[3] = {19, 7, 0};
    const int widths[3] = {12, 12, 7};
    for (int lv = 0; lv < 3; ++lv) {
      const int shf = shifts[lv];
      const u32 nbm = (1u << widths[lv]) - 1u;
      __syncthreads();
      for (int i = tid; i < kBins; i += blockDim.x) sh.hist[i] = 0;
      __syncthreads();
      for (int64_t base = c0; base < c1; base += 4 * (int64_t)blockDim.x) {  // whole warps iterate: the increments are aggregated
        const int64_t j4 = base + 4 * tid;
        u32 key[4];
        dense_keys4(p, n, j4, c1, key);
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const bool in = j4 + q < c1 && (lv == 0 || (key[q] >> (shf + widths[lv])) == prefix);
          hist_add_aggregated(sh.hist, in, (key[q] >> shf) & nbm);  // rows that end up here are full of equal digits
        }
      }
      __syncthreads();
      flush_hist(sh.hist, ghist + (1 + lv) * kBins, kBins);
      cl.sync();
      u32 b, above, total;
      load_and_find(sh, ghist + (1 + lv) * kBins, need, &b, &above, &total);
      if (b == kFull) { bad = true; b = 0; above = 0; }
      need -= above;
      prefix = (prefix << widths[lv]) | b;
    }
    const u32 T = prefix;          // key of the k-th largest score
    const u32 n_gt = k - need;     // entries strictly above it; `need` ties are to be taken
    // entries above T in any order, and this block's count of ties
    u32 my_ties = 0;
    for (int64_t base = c0; base < c1; base += 4 * (int64_t)blockDim.x) {
      const int64_t j4 = base + 4 * tid;
      u32 key[4];
      dense_keys4(p, n, j4, c1, key);
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const bool gt = j4 + q < c1 && key[q] > T;
        my_ties += (j4 + q < c1 && key[q] == T) ? 1u : 0u;
        const u32 pos = warp_reserve_global(gt, &ctl->acount);
        if (gt && pos < n_gt) Wl[pos] = make_composite(key[q], (u32)(j4 + q));
      }
    }
    u32 block_ties;
    block_excl_scan(my_ties, sh.scan, &block_ties);
    if (tid == 0) btot[kMaxCluster + rk] = block_ties;
    cl.sync();
    u32 taken = 0, all_ties = 0;  // ties in lower-index blocks, and in the whole row
    for (u32 c = 0; c < CS; ++c) {
      const u32 t = __ldcg(&btot[kMaxCluster + c]);
      if (c < rk) taken += t;
      all_ties += t;
    }
    if (all_ties < need) bad = true;
    // ties in index order: the first `need` of them
    for (int64_t base = c0; base < c1 && taken < need; base += 4 * (int64_t)blockDim.x) {
      const int64_t j4 = base + 4 * tid;  // threads hold consecutive quads: thread order is index order
      u32 key[4];
      dense_keys4(p, n, j4, c1, key);
      u32 mine = 0;
#pragma unroll
      for (int q = 0; q < 4; ++q) mine += (j4 + q < c1 && key[q] == T) ? 1u : 0u;
      u32 total;
      u32 rank = taken + block_excl_scan(mine, sh.scan, &total);
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        if (j4 + q < c1 && key[q] == T) {
          if (rank < need && RT_INB(n_gt + rank < k)) Wl[n_gt + rank] = make_composite(T, (u32)(j4 + q));
          ++rank;
        }
      }
      taken += total;
    }
    cl.sync();  // winner list complete
    if (rk == 0 && tid == 0 && (bad || __ldcg(&ctl->acount) != n_gt)) atomicOr(&p.gctl->err, kErrDenseSelect);
    if (!bad)
      for (u32 i = first_t; i < k; i += stride_t) set_winner(mask, composite_idx(__ldcg(&Wl[i])), p.d);
    cl.sync();  // every winner bit is set
  }
  if (p.wide) {  // k_wide_prefix and k_wide_emit take over
    if (rk == 0 && tid == 0) ctl->took_dense = took_dense ? 1u : 0u;
    return;
  }

  // ---- emission.  The rank of a winner (its place in the ascending output) is the number of mask
  //      bits before it.  (E1) every warp of the cluster owns a fixed segment of the mask row and
  //      writes, per quad (four words, 128 coordinates), the bits before it inside the segment;
  //      (E2) the segment totals are exchanged and scanned; (E3) every candidate whose mask bit is
  //      set looks its rank up (segment base + quad prefix + bits before it in the quad) and writes
  //      its pair there.  Work in E3 follows the candidate lists, which are spread evenly over the
  //      threads, so a region dense with winners costs no more than a sparse one. ----
  __syncthreads();
  const int lane = tid & 31, warp = tid >> 5;
  post_prefix_segment(p, n, rk * (u32)nw + (u32)warp, seg_units, lane);
  cl.sync();  // (3) segment totals and quad prefixes of the whole row are written
  u32* s_segbase = sh.spare;  // kMaxSegments <= kBins entries
  {
    u32 total;
    const u32 t = (u32)tid < nseg ? __ldcg(&p.segtot[(size_t)n * kMaxSegments + tid]) : 0u;
    const u32 base = block_excl_scan(t, sh.scan, &total);
    if ((u32)tid < nseg) {
      s_segbase[tid] = base;
      if (rk == 0) p.segbase[(size_t)n * kMaxSegments + tid] = base;  // for k_aggregate
    }
    __syncthreads();
    if (total != k) {  // the same in every block
      if (rk == 0 && tid == 0) atomicOr(&p.gctl->err, kErrCountMismatch);
      return;
    }
  }
  post_emit(p, n, first_t, stride_t, ncand, novr, took_dense, cutoff, bshift, b1, s_segbase, seg_units);
}

// ---------------------------------------------------------------------------------------------
// Wide mode (N*k large): the list phases of k_post as kernels of their own on the whole grid, blockIdx.y
// = worker, because there the lists are long enough for throughput, not latency, to decide:
//   k_wide_hist -> k_wide_classify -> k_post (refinement or dense path only) -> k_wide_prefix -> k_wide_emit.
// The mask row is cut into kMaxSegments segments whatever the grid.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kBlockPost, 1024 / kBlockPost) k_wide_hist(PostArgs p) {
  __shared__ u32 s_hist[kBins];
  grid_dependency_begin();
  const int n = blockIdx.y, tid = threadIdx.x;
  const u32 stride_t = gridDim.x * blockDim.x, first_t = blockIdx.x * blockDim.x + tid;
  const WorkerCtl* ctl = p.ctl + n;
  const u32 cutoff = ctl->cutoff, bshift = ctl->bin_shift, cand_count = ctl->cand_count;
  const bool dense = ctl->force_dense != 0;
  const u32 ncand = (u64)cand_count > (u64)p.capA ? (u32)p.capA : cand_count;
  for (int i = tid; i < kBins; i += blockDim.x) s_hist[i] = 0;
  for (u32 i = first_t; i < (u32)kSampleBins; i += stride_t) p.shist[(size_t)n * kSampleBins + i] = 0;
  __syncthreads();
  post_sweep(p, n, first_t, stride_t, dense, ncand, cutoff, bshift, s_hist);
  __syncthreads();
  if (!dense) flush_hist(s_hist, p.ghist + (size_t)n * 4 * kBins, kBins);
}

__global__ void __launch_bounds__(kBlockPost, 1024 / kBlockPost) k_wide_classify(PostArgs p) {
  __shared__ __align__(16) PostShared sh;
  grid_dependency_begin();
  const int n = blockIdx.y, tid = threadIdx.x;
  const u32 stride_t = gridDim.x * blockDim.x, first_t = blockIdx.x * blockDim.x + tid;
  WorkerCtl* ctl = p.ctl + n;
  const u32 cutoff = ctl->cutoff, bshift = ctl->bin_shift, cand_count = ctl->cand_count;
  bool dense = ctl->force_dense != 0;
  const bool overflow = (u64)cand_count > (u64)p.capA;
  const u32 ncand = overflow ? (u32)p.capA : cand_count;
  u32 b1 = kFull, above1 = 0, nvalid = 0;
  if (!dense) {  // every block finds the threshold bin by itself (all get the same answer)
    load_and_find(sh, p.ghist + (size_t)n * 4 * kBins, (u32)p.k, &b1, &above1, &nvalid);
    if (b1 == kFull || overflow) dense = true;
  }
  if (blockIdx.x == 0 && tid == 0) {
    ctl->b1 = b1;
    ctl->above1 = above1;
    ctl->go_dense = dense ? 1u : 0u;
    ctl->n_valid = nvalid;
    if (dense && ctl->force_dense == 0) ask_for_exact_cutoffs(&ctl->exact_rounds, &ctl->exact_window);
  }
  if (!dense) post_classify(p, n, first_t, stride_t, ncand, p.use_marks ? (u32)p.k : 0u, cutoff, bshift, b1);
}

__global__ void __launch_bounds__(kBlockPost, 1024 / kBlockPost) k_wide_prefix(PostArgs p) {
  grid_dependency_begin();
  const int n = blockIdx.y;
  const int lane = threadIdx.x & 31, nw = blockDim.x >> 5;
  const int64_t U = p.W >> 3;
  const int64_t seg_units = (U + kMaxSegments - 1) / kMaxSegments;
  for (u32 seg = blockIdx.x * nw + (threadIdx.x >> 5); seg < (u32)kMaxSegments; seg += gridDim.x * nw)
    post_prefix_segment(p, n, seg, seg_units, lane);
}

__global__ void __launch_bounds__(kBlockPost, 1024 / kBlockPost) k_wide_emit(PostArgs p) {
  __shared__ u32 s_segbase[kMaxSegments];
  __shared__ u32 s_scan[33];
  grid_dependency_begin();
  const int n = blockIdx.y, tid = threadIdx.x;
  const u32 stride_t = gridDim.x * blockDim.x, first_t = blockIdx.x * blockDim.x + tid;
  const WorkerCtl* ctl = p.ctl + n;
  const u32 cutoff = ctl->cutoff, bshift = ctl->bin_shift, cand_count = ctl->cand_count;
  const u32 b1 = ctl->b1;
  const bool took_dense = ctl->took_dense != 0;
  const u32 ncand = (u64)cand_count > (u64)p.capA ? (u32)p.capA : cand_count;
  const int64_t U = p.W >> 3;
  const int64_t seg_units = (U + kMaxSegments - 1) / kMaxSegments;
  u32 total;
  const u32 t = tid < kMaxSegments ? __ldcg(&p.segtot[(size_t)n * kMaxSegments + tid]) : 0u;
  const u32 base = block_excl_scan(t, s_scan, &total);  // blockDim.x >= kMaxSegments
  if (tid < kMaxSegments) {
    s_segbase[tid] = base;
    if (blockIdx.x == 0) p.segbase[(size_t)n * kMaxSegments + tid] = base;  // for k_aggregate
  }
  __syncthreads();
  if (total != (u32)p.k) {
    if (blockIdx.x == 0 && tid == 0) atomicOr(&p.gctl->err, kErrCountMismatch);
    return;
  }
  post_emit(p, n, first_t, stride_t, ncand, p.use_marks ? (u32)p.k : 0u, took_dense, cutoff, bshift, b1, s_segbase,
            seg_units);
}

// After k_post in pair mode: (index, value) pairs, in rank order in the workers' B lists, go to the
// caller's arrays and to the library's own copy.
struct UnzipArgs {
  const u64* candB;
  int64_t stride;
  int64_t k;
  int N;
  int32_t* out_idx;
  float* out_val;
  int32_t* cur_idx;
  float* cur_val;
};

__global__ void __launch_bounds__(256) k_unzip(UnzipArgs p) {
  grid_dependency_begin();
  const int n = blockIdx.y;
  const uint2* pairs = reinterpret_cast<const uint2*>(p.candB + (size_t)n * p.stride);
  const size_t obase = (size_t)n * p.k;
  for (int64_t r = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; r < p.k; r += (int64_t)gridDim.x * blockDim.x) {
    const uint2 v = __ldcs(pairs + r);
    p.out_idx[obase + r] = (int32_t)v.x;
    p.cur_idx[obase + r] = (int32_t)v.x;
    p.out_val[obase + r] = __uint_as_float(v.y);
    p.cur_val[obase + r] = __uint_as_float(v.y);
  }
}

// ---------------------------------------------------------------------------------------------
// k_dense: exact selection straight from the rows, by the whole grid (a cooperative launch; the phases are
// separated by grid-wide barriers).  It serves the workers whose candidate path gave up (ctl->go_dense:
// cutoff guessed too high, list overflowed, or the dense path was asked for) and every worker in
// layer-wise mode, where each layer of a row is a selection problem of its own: a row is a sequence of
// segments (one for the whole row in the plain mode), segment s keeps its k_s largest (score, lowest index).
//
// Per segment:
//   (A) a histogram of the top 12 key bits over the segment's part of the row, restricted to keys at or above
//       a lower bound `lo` (a hint: the sampled cutoff, or in layer-wise mode the bound that the segment's last
//       selection left: the key of the entry max(k_s, 32) places below its threshold), so that nearly all
//       entries cost a compare and no shared-memory atomic.  From the top down, the bin b0 that
//       holds the k_s-th largest, the entries above it and the number c0 inside it.  If the histogram holds
//       fewer than k_s entries the hint was too high and the pass is repeated for that segment with lo an octave
//       lower, and if need be a third time with lo = 0.
//   (B) a second pass over the rows: entries above bin b0 are winners (mask bit set, composite appended to
//       the worker's winner list); the c0 entries inside it go to a list of their own,
//   (C) from which one block takes the `need` largest composites (key, lowest index).
// In layer-wise mode the streaming pass has already gathered every entry at or above its segment's bound into the
// worker's candidate list; (A) and (B) of such a segment read that list instead of the rows.
// A segment whose bin b0 does not fit the list space (error feedback has packed thousands of entries into it, or
// the row is full of equal values) stays on the rows for a second digit of 12 bits.  If its bin, 4096 times
// narrower, fits, the segment goes the list way from there ((B) and (C) with 24 bits fixed).  Otherwise a third
// digit of 7 bits gives the threshold key T and the number of entries equal to T that are to be taken; if there
// are more of those than needed, their counts per tile are scanned so that the lowest indices win; a last pass
// over the rows sets the winners.
// Rows are cut into tiles of kDenseTile coordinates that never straddle a segment; a block owns a
// contiguous run of tiles.  If nobody needs the path the kernel returns at once.
// ---------------------------------------------------------------------------------------------
constexpr int kDenseThreads = 512;
constexpr int kDenseUnroll = 4;   // quads a thread has in flight: 64 bytes, 64 KB per SM with two blocks of 512 threads
constexpr int kDenseTile = kDenseUnroll * 4 * kDenseThreads;  // 8192 coordinates: one step of the walk
constexpr int kDenseWarps = kDenseThreads / 32;
constexpr int kDenseMaxFlagged = 1024;
constexpr u32 kOctave = 0x00800000u;  // one binary order of magnitude in key units
constexpr u32 kHintMargin = 2u << 19;  // two bins of the first digit (an eighth of an octave)

enum : u32 { kSegList = 0u, kSegRows = 1u, kSegRetry = 2u, kSegList2 = 3u,
             kSegWant = 4u,    // first digit found, list space not yet dealt out (only inside the first-digit search)
             kSegZero = 5u };  // every key of the segment is zero (a layer without gradient): its lowest k_s indices win
enum : u32 { kFlagRetry = 1u, kFlagRows = 2u, kFlagOrdered = 4u, kFlagBad = 8u, kFlagRows2 = 16u,
            kFlagWalk = 32u };  // layer-wise mode: some segment takes its first digit from the rows (otherwise no block walks its tiles for it)

struct __align__(16) SegState {
  u32 prefix;  // digits of the threshold key fixed so far
  u32 need;    // entries still to be taken among those that match the prefix
  u32 ties;    // entries in the bin of the last digit found (after the last digit: entries equal to the threshold key)
  u32 mode;    // kSegList, kSegRows, or kSegRetry while the first digit has to be counted again
  u32 lo;      // keys below this are left out of the first histogram
  u32 boff;    // kSegList: where the segment's in-bin list starts in the worker's B list
  u32 bfill;   //           entries written there so far
  u32 sh;      // key bits below the digits in `prefix` (19 after the first digit, 7 after the second)
  u32 src;     // 1: the first digit and the compaction read the worker's candidate list (layer-wise mode: the streaming
               //    pass gathered every entry at or above the segment's bound); 0: they walk the rows
  u32 nonzero; // set by the first digit's walk when it saw a key other than zero (or did not look: a bound was set)
  u32 pad[2];
};

struct DenseArgs {
  PostArgs p;
  int N;
  int n_seg;
  int finish;               // also rank the winners and emit the pairs (otherwise k_wide_prefix / k_wide_emit follow)
  int layered;              // hints come from last round's thresholds (seg_thr), not from the sampled cutoff
  u32 emit_segments;        // mask-row segments the emission and k_aggregate use
  int64_t tiles;            // tiles per worker
  const int64_t* seg_end;   // [n_seg] end of each segment (ascending, the last is d)
  const int64_t* seg_kpre;  // [n_seg + 1] exclusive prefix sums of the segments' k
  const int64_t* seg_tile0; // [n_seg + 1] first tile of each segment
  u32* dhist;               // [N][n_seg][kBins], all zero between launches
  SegState* seg;            // [N][n_seg]
  u32* seg_thr;             // [N][n_seg] the lower bound the last round left for this one (see leave_rank_bound; 0: none)
  u32* tile_ties;           // [N][tiles][2]: entries equal to the threshold key in the tile, and in lower tiles of the segment
};

__device__ __forceinline__ int dense_seg_of_tile(const int64_t* seg_tile0, int n_seg, int64_t t) {
  int lo = 0, hi = n_seg;  // the last segment whose first tile is at or before t
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (seg_tile0[mid] <= t) lo = mid; else hi = mid;
  }
  return lo;
}

// Calls f(j4, key, in) with the score keys of the quad j4 .. j4 + 3 (in[q]: the entry lies in [t0, t1)) for the
// quads that meet [t0, t1), but only where some lane of the warp holds a key of at least min_key in its quad: the
// call is made by all lanes of such a warp or by none, so f may use warp-wide primitives, and with min_key == 0 it
// is made by every thread of the block the same number of times, so f may then use block-wide ones.  With
// PER_THREAD only the threads whose own quad holds such a key call f (which must then do without warp-wide
// primitives), and every lane calls after() once per step of the loop (kDenseUnroll quads), converged.  A thread's
// quads within one step of the loop are 4 * blockDim.x coordinates apart, and threads hold consecutive quads.
// kDenseUnroll 16-byte loads per thread are in flight.  Keys as in dense_key: the regularised score on the previous
// support, bits(|a|) elsewhere.  With SKIP_MARKED the walk does not look at the previous support at all (no mask
// word per quad, no binary search for a score: a chain of dependent loads that stalls the warp): every key is
// bits(|a|); the caller sorts the previous support out afterwards (entries staged for a list are tested against
// the old mask in batches when the list is written out; a histogram is corrected from the override list, which
// holds those entries' scores in index order).
struct NoHook { __device__ __forceinline__ void operator()() const {} };

template <bool SKIP_MARKED, bool PER_THREAD = false, typename F, typename G = NoHook>
__device__ __forceinline__ void dense_walk(const PostArgs& p, int n, int64_t t0, int64_t t1, u32 min_key, F f, G after = G()) {
  const float* row = p.eps + (size_t)n * p.ld;
  const u32* marks = (p.use_marks && !SKIP_MARKED) ? p.mask_old + (size_t)n * p.W : nullptr;
  constexpr int kU = kDenseUnroll;
  const int stride = 4 * (int)blockDim.x;
  for (int64_t base = t0 & ~(int64_t)3; base < t1; base += kU * stride) {
    // this step's part of [t0, t1) as offsets from base
    const int lo_off = (int)(t0 - base);  // <= 3; negative after the first step
    const int hi_off = t1 - base < (int64_t)kU * stride ? (int)(t1 - base) : kU * stride;
    float4 e[kU];
    u32 w[kU];
#pragma unroll
    for (int u = 0; u < kU; ++u) {
      const int off = u * stride + 4 * (int)threadIdx.x;
      const bool live = off < hi_off;  // rows are padded to a multiple of 1024: the whole quad is inside the row's storage
      e[u] = live ? __ldcs(reinterpret_cast<const float4*>(row + base + off)) : make_float4(0.f, 0.f, 0.f, 0.f);
      w[u] = (live && marks) ? (__ldg(marks + ((base + off) >> 5)) >> ((base + off) & 31)) & 15u : 0u;
    }
#pragma unroll
    for (int u = 0; u < kU; ++u) {
      if (u * stride >= hi_off) break;  // the same in every thread
      const int off = u * stride + 4 * (int)threadIdx.x;
      const int64_t j4 = base + off;
      u32 key[4] = {__float_as_uint(e[u].x) & 0x7FFFFFFFu, __float_as_uint(e[u].y) & 0x7FFFFFFFu,
                    __float_as_uint(e[u].z) & 0x7FFFFFFFu, __float_as_uint(e[u].w) & 0x7FFFFFFFu};
      bool in[4] = {true, true, true, true};
      if (w[u] != 0u || off < lo_off || off + 4 > hi_off) {  // rare: an entry of the previous support, or a quad across an end
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          in[q] = off + q >= lo_off && off + q < hi_off;
          if (!in[q]) key[q] = 0u;
          else if ((w[u] >> q) & 1u) key[q] = dense_key(p, n, j4 + q);
        }
      }
      const u32 top = max(max(key[0], key[1]), max(key[2], key[3]));
      if (PER_THREAD) {  // f by the threads concerned only (no warp-wide primitive in it)
        if (top >= min_key) f(j4, key, in);
      } else if (__any_sync(kFull, top >= min_key)) {
        f(j4, key, in);
      }
    }
    if (PER_THREAD) {  // the hook by all lanes, converged, once per step
      __syncwarp();
      after();
    }
  }
}

__device__ __forceinline__ int dense_seg_of_index(const int64_t* seg_end, int n_seg, int64_t j) {
  int lo = 0, hi = n_seg - 1;  // the first segment whose end lies beyond j
  while (lo < hi) {
    const int mid = (lo + hi) >> 1;
    if (seg_end[mid] <= j) lo = mid + 1; else hi = mid;
  }
  return lo;
}

// Layer-wise mode, before the streaming pass: the candidate cutoff of every span of kCutSpan coordinates, i.e. the
// lowest of the bounds that the last round left for the layers the span meets (seg_thr; a layer without one admits
// nothing, 0xFFFFFFFF, and is selected from the rows).  The streaming pass then compacts, per worker, every entry that
// can matter to its layer, and k_dense takes the layers' first histogram and their winners from that list instead
// of from two more passes over the rows.
__global__ void __launch_bounds__(256) k_layer_cutoffs(u32* chunk_cut, int64_t cuts, int64_t d, int N, int n_seg,
                                                       const int64_t* seg_end, const u32* seg_thr) {
  grid_dependency_begin();
  const int64_t total = cuts * N;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    const int n = (int)(i / cuts);
    const int64_t c = i - (int64_t)n * cuts;
    const int64_t j0 = c * kCutSpan, j1 = j0 + kCutSpan < d ? j0 + kCutSpan : d;
    u32 cut = kFull;
    for (int s = dense_seg_of_index(seg_end, n_seg, j0); s < n_seg; ++s) {
      const u32 thr = seg_thr[(size_t)n * n_seg + s];
      const u32 lo = thr ? thr : kFull;
      cut = lo < cut ? lo : cut;
      if (seg_end[s] >= j1) break;
    }
    chunk_cut[i] = cut;
  }
}

__device__ __forceinline__ SegState load_seg(const DenseArgs& a, int n, int s) {  // written by other blocks of this launch
  const uint4* q = reinterpret_cast<const uint4*>(a.seg + (size_t)n * a.n_seg + s);
  const uint4 v = __ldcg(q), x = __ldcg(q + 1), y = __ldcg(q + 2);
  SegState r;
  r.prefix = v.x; r.need = v.y; r.ties = v.z; r.mode = v.w;
  r.lo = x.x; r.boff = x.y; r.bfill = x.z; r.sh = x.w;
  r.src = y.x; r.nonzero = y.y; r.pad[0] = r.pad[1] = 0u;
  return r;
}

// Take `want` entries of a list of `cap` whose fill counter is *fill, but only if they fit: the counter never
// passes cap, so space that was granted is never granted twice.  One thread; at most a few retries under contention.
__device__ __forceinline__ bool reserve_list_space(u32* fill, u32 want, u64 cap, u32* off) {
  u32 cur = *reinterpret_cast<volatile u32*>(fill);
  for (int tries = 0; tries < 1024; ++tries) {
    if ((u64)cur + want > cap) return false;
    const u32 seen = atomicCAS(fill, cur, cur + want);
    if (seen == cur) {
      *off = cur;
      return true;
    }
    cur = seen;
  }
  return false;  // (gives up: the segment then takes the way that needs no list)
}

// The tile `w` of the run of tiles the flagged workers have together: worker, segment and index range.
struct DenseTile {
  int n, s;
  int64_t t;       // tile number inside the worker's row
  int64_t t0, t1;  // coordinates
};

__device__ __forceinline__ DenseTile dense_tile(const DenseArgs& a, const u32* s_flagged, int64_t w) {
  DenseTile r;
  const int64_t f = w / a.tiles;
  r.n = (int)s_flagged[f];
  r.t = w - f * a.tiles;
  r.s = dense_seg_of_tile(a.seg_tile0, a.n_seg, r.t);
  const int64_t begin = r.s ? a.seg_end[r.s - 1] : 0;
  r.t0 = begin + (r.t - a.seg_tile0[r.s]) * kDenseTile;
  r.t1 = r.t0 + kDenseTile < a.seg_end[r.s] ? r.t0 + kDenseTile : a.seg_end[r.s];
  return r;
}

// Drop from a warp's list the entries whose index is set in `marks` (the previous support): the probes are issued
// four per lane at a time, so the warp waits for memory a few times per call, not once per entry.  Returns the
// number kept (compacted to the front, order preserved).
__device__ __forceinline__ u32 warp_drop_marked(u64* list, u32 total, const u32* marks, int lane) {
  u32 kept = 0;
#pragma unroll 1
  for (u32 r0 = 0; r0 < total; r0 += 128) {
    u64 ent[4];
    u32 word[4];
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const u32 i = r0 + (u32)r * 32 + lane;
      ent[r] = i < total ? list[i] : 0ull;
      word[r] = i < total ? __ldg(&marks[composite_idx(ent[r]) >> 5]) : 0u;
    }
    __syncwarp();  // every lane has read its entries before any is overwritten
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const u32 i = r0 + (u32)r * 32 + lane;
      const bool keep = i < total && !((word[r] >> (composite_idx(ent[r]) & 31)) & 1u);
      const u32 m = __ballot_sync(kFull, keep);
      if (keep) list[kept + __popc(m & ((1u << lane) - 1u))] = ent[r];  // kept <= r0 + 32 r: behind the reads
      kept += __popc(m);
    }
    __syncwarp();
  }
  return kept;
}

// A warp's staging list in shared memory (kWarpList composites): entries are added in ballot order and written out
// to a global list, whose fill counter one lane advances, before the list can overflow.
__device__ __forceinline__ void stage_add(u64* list, u32& count, bool pred, u64 value, int lane) {
  const u32 m = __ballot_sync(kFull, pred);
  if (pred && RT_INB(count + __popc(m & ((1u << lane) - 1u)) < (u32)kWarpList))
    list[count + __popc(m & ((1u << lane) - 1u))] = value;
  count += __popc(m);
}

__device__ __forceinline__ void stage_flush(u64* list, u32& count, u32* fill, u64* dst, u64 cap, int lane) {
  __syncwarp();
  if (count) {
    u32 base = 0;
    if (lane == 0) base = atomicAdd(fill, count);
    base = __shfl_sync(kFull, base, 0);
    for (u32 i = lane; i < count; i += 32)
      if (RT_INB((u64)base + i < cap)) dst[(u64)base + i] = list[i];
  }
  count = 0;
  __syncwarp();
}

// LAYERED: layer-wise mode (hints from last round's segments, segments fed from the candidate list); the plain
// instance carries none of that code.
template <bool LAYERED>
__global__ void __launch_bounds__(kDenseThreads, 2) k_dense(DenseArgs a) {
  extern __shared__ __align__(16) u64 s_stage[];  // [kDenseWarps][2 * kWarpList]: per-warp staging lists
  __shared__ __align__(16) u32 s_hist[kBins];
  __shared__ u32 s_flagged[kDenseMaxFlagged];
  __shared__ u32 s_cbase[kDenseMaxFlagged + 1];  // layer-wise mode: 32-entry pieces of the candidate lists before each flagged worker's
  __shared__ u32 s_scan[33];
  __shared__ u32 s_res[4];
  __shared__ u32 s_cnt, s_nf, s_nf2, s_nz;
  __shared__ u64 s_T;
  __shared__ u32 s_wcnt[1][kDenseWarps];
  cg::grid_group grid = cg::this_grid();
  const PostArgs& p = a.p;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const u32 k = (u32)p.k;
  u64* listA = s_stage + (size_t)warp * 2 * kWarpList;  // this warp's staging space: 2 * kWarpList entries

  for (int g0 = 0; g0 < a.N; g0 += kDenseMaxFlagged) {  // groups of workers; the flags are the same in every block
    {  // the flagged workers of this group, in order
      constexpr int kPer = kDenseMaxFlagged / kDenseThreads;  // consecutive workers per thread
      u32 fl = 0, cnt = 0;
#pragma unroll
      for (int i = 0; i < kPer; ++i) {
        const int n = g0 + kPer * tid + i;
        if (n < a.N && p.ctl[n].go_dense) { fl |= 1u << i; ++cnt; }
      }
      u32 total;
      u32 at = block_excl_scan(cnt, s_scan, &total);
#pragma unroll
      for (int i = 0; i < kPer; ++i)
        if ((fl >> i) & 1u) s_flagged[at++] = (u32)(g0 + kPer * tid + i);
      if (tid == 0) s_nf = total;
      __syncthreads();
    }
    const int64_t nf = s_nf;
    if (nf == 0) continue;  // the same decision in every block: no barrier is skipped by some and taken by others
    const int64_t total_tiles = nf * a.tiles;
    const int64_t per = (total_tiles + gridDim.x - 1) / gridDim.x;
    const int64_t w_begin = (int64_t)blockIdx.x * per < total_tiles ? (int64_t)blockIdx.x * per : total_tiles;
    const int64_t w_end = w_begin + per < total_tiles ? w_begin + per : total_tiles;
    const int64_t nsegs = nf * a.n_seg;
    // The two walks of the first digit take the tiles in runs: one contiguous run per block in the plain mode; in
    // layer-wise mode runs of 16 tiles dealt round-robin, because there the tiles to be walked (layers without a bound,
    // layers without gradient) lie in clusters that contiguous runs would leave to a few blocks.
    const int64_t t_run = LAYERED ? 16 : per;
    const int64_t t_step = LAYERED ? (int64_t)gridDim.x * 16 : (total_tiles > 0 ? total_tiles : 1);
    if (LAYERED) {  // (a worker whose list overflowed has no pieces: none of its segments is fed from the list)
      constexpr int kPer = kDenseMaxFlagged / kDenseThreads;
      u32 mine[kPer], sum = 0, total;
#pragma unroll
      for (int i = 0; i < kPer; ++i) {
        const int64_t f = kPer * tid + i;
        u32 cc = 0;
        if (f < nf) cc = p.ctl[s_flagged[f]].cand_count;
        mine[i] = (u64)cc <= (u64)p.capA ? (cc + 31u) >> 5 : 0u;
        sum += mine[i];
      }
      u32 at = block_excl_scan(sum, s_scan, &total);
#pragma unroll
      for (int i = 0; i < kPer; ++i) {
        s_cbase[kPer * tid + i] = at;
        at += mine[i];
      }
      if (tid == 0) s_cbase[kDenseMaxFlagged] = total;
      __syncthreads();
    }

    // One histogram pass over this block's tiles.  which(seg state) says whether a segment takes part; the entries
    // counted are those with key >= lo (first digit) or whose higher digits equal the prefix (later digits).
    auto hist_pass = [&](int lv, u32 want_mode, bool walk) {
      const int shf = lv == 0 ? 19 : (lv == 1 ? 7 : 0);  // digits of 12, 12 and 7 bits
      const int width = lv == 2 ? 7 : 12;
      const u32 nbm = (1u << width) - 1u;
      int cur_n = -1, cur_s = -1;
      bool dirty = false;
      SegState st;
      st.mode = ~0u;
      for (int i = tid; i < kBins; i += blockDim.x) s_hist[i] = 0;
      if (tid == 0) s_nz = 0u;
      __syncthreads();
      for (int64_t c0 = walk ? (int64_t)blockIdx.x * t_run : total_tiles; c0 < total_tiles; c0 += t_step)
      for (int64_t w = c0, c1 = c0 + t_run < total_tiles ? c0 + t_run : total_tiles; w < c1; ++w) {
        const DenseTile t = dense_tile(a, s_flagged, w);
        if (t.n != cur_n || t.s != cur_s) {
          if (dirty) {
            __syncthreads();
            flush_hist(s_hist, a.dhist + ((size_t)cur_n * a.n_seg + cur_s) * kBins, kBins);
            // (with a bound the walk did not look at every entry: the segment is not known to be all zero)
            if (lv == 0 && tid == 0 && (s_nz || st.lo != 0u)) atomicOr(&a.seg[(size_t)cur_n * a.n_seg + cur_s].nonzero, 1u);
            __syncthreads();
            for (int i = tid; i < kBins; i += blockDim.x) s_hist[i] = 0;
            if (tid == 0) s_nz = 0u;
            __syncthreads();
            dirty = false;
          }
          cur_n = t.n; cur_s = t.s;
          st = load_seg(a, t.n, t.s);  // nothing writes it during this pass
        }
        if (st.mode != want_mode || (LAYERED && lv == 0 && st.src)) { w += a.seg_tile0[t.s + 1] - 1 - t.t; continue; }  // nothing to do in this segment: on to its last tile (the same in every thread of the block)
        dirty = true;
        const u32 floor_key = lv == 0 ? st.lo : st.prefix << (shf + width);  // no entry below it is counted
        auto count = [&](int64_t j4, const u32 (&key)[4], const bool (&in)[4]) {
          bool use[4];
#pragma unroll
          for (int q = 0; q < 4; ++q)
            use[q] = in[q] && (lv == 0 ? key[q] >= st.lo : (key[q] >> (shf + width)) == st.prefix);
#pragma unroll
          for (int q = 0; q < 4; ++q) hist_add_aggregated(s_hist, use[q], (key[q] >> shf) & nbm);
        };
        if (lv == 0 && st.lo != 0u) {
          // with a lower bound few entries count: the threads that hold one add it themselves
          dense_walk<true, true>(p, t.n, t.t0, t.t1, floor_key, [&](int64_t j4, const u32 (&key)[4], const bool (&in)[4]) {
#pragma unroll
            for (int q = 0; q < 4; ++q)
              if (in[q] && key[q] >= st.lo) atomicAdd(&s_hist[key[q] >> 19], 1u);
          });
        } else if (lv == 0) {
          u32 seen = 0;  // (the previous support is counted from the override list; its scores are zero where |a| is)
          dense_walk<true>(p, t.n, t.t0, t.t1, floor_key, [&](int64_t j4, const u32 (&key)[4], const bool (&in)[4]) {
            // 128 equal keys (a stretch without gradient) are counted with one addition
            const u32 v = __shfl_sync(kFull, key[0], 0);
            const bool same = in[0] && in[1] && in[2] && in[3] && key[0] == v && key[1] == v && key[2] == v && key[3] == v;
            if (__all_sync(kFull, same)) {
              if (lane == 0) atomicAdd(&s_hist[v >> 19], 128u);
            } else {
              count(j4, key, in);
            }
#pragma unroll
            for (int q = 0; q < 4; ++q) seen |= in[q] ? key[q] : 0u;
          });
          if (seen) s_nz = 1u;
        } else {
          dense_walk<false>(p, t.n, t.t0, t.t1, floor_key, count);
        }
      }
      __syncthreads();
      if (dirty) {
        flush_hist(s_hist, a.dhist + ((size_t)cur_n * a.n_seg + cur_s) * kBins, kBins);
        if (lv == 0 && tid == 0 && (s_nz || st.lo != 0u)) atomicOr(&a.seg[(size_t)cur_n * a.n_seg + cur_s].nonzero, 1u);
      }
      if (LAYERED && lv == 0) {
        // Layer-wise mode: the candidate lists of the segments fed from them, and the entries of the previous
        // support (override list), as one run of 32-entry tasks over all flagged workers, dealt to the warps of the
        // grid in contiguous pieces.  The segment ends and the segments' bounds are looked up in shared memory
        // (the staging space, not used in this pass) when they fit there.
        u32* t_end = reinterpret_cast<u32*>(s_stage);  // [n_seg]
        u32* t_lo = t_end + a.n_seg;                   // [nsegs]: bound (keys have 31 bits) | list-fed << 31, or kFull if the segment takes no part
        const bool fast = (u64)nsegs + (u64)a.n_seg <= (u64)kDenseWarps * 2u * kWarpList * 2u;
        if (fast) {
          for (int i = tid; i < a.n_seg; i += blockDim.x) t_end[i] = (u32)a.seg_end[i];
          for (int64_t v = tid; v < nsegs; v += blockDim.x) {
            const SegState sg = load_seg(a, (int)s_flagged[v / a.n_seg], (int)(v % a.n_seg));
            t_lo[v] = sg.mode == want_mode ? (sg.lo | (sg.src << 31)) : kFull;
          }
          __syncthreads();
        }
        auto seg_of = [&](u32 j) -> int {
          if (!fast) return dense_seg_of_index(a.seg_end, a.n_seg, (int64_t)j);
          int lo = 0, hi = a.n_seg - 1;  // the first segment whose end lies beyond j
          while (lo < hi) {
            const int mid = (lo + hi) >> 1;
            if (t_end[mid] <= j) lo = mid + 1; else hi = mid;
          }
          return lo;
        };
        auto bound_of = [&](int64_t f, int n, int s) -> u32 {
          if (fast) return t_lo[f * a.n_seg + s];
          const SegState sg = load_seg(a, n, s);
          return sg.mode == want_mode ? (sg.lo | (sg.src << 31)) : kFull;
        };
        const int64_t gw = (int64_t)warp * gridDim.x + blockIdx.x, nwarps = (int64_t)gridDim.x * kDenseWarps;  // warps numbered across the blocks: a short run of tasks spreads over all SMs
        {  // candidates
          const int64_t tasks = s_cbase[nf];
          const int64_t per = (tasks + nwarps - 1) / nwarps;
          const int64_t t0 = gw * per, t1 = t0 + per < tasks ? t0 + per : tasks;
          int64_t f = 0;
          if (t0 < t1) {
            int64_t lo = 0, hi = nf;  // the worker whose tasks include t0
            while (hi - lo > 1) {
              const int64_t mid = (lo + hi) >> 1;
              if ((int64_t)s_cbase[mid] <= t0) lo = mid; else hi = mid;
            }
            f = lo;
          }
          auto fetch = [&](int64_t t, int64_t& ff, bool& live) -> u64 {
            live = false;
            if (t >= t1) return 0ull;
            while (t >= (int64_t)s_cbase[ff + 1]) ++ff;
            const int n = (int)s_flagged[ff];
            const int64_t i = (t - (int64_t)s_cbase[ff]) * 32 + lane;
            live = i < (int64_t)p.ctl[n].cand_count;
            return live ? __ldcg(p.candA + (size_t)n * p.stride + i) : 0ull;
          };
          int64_t f_next = f;
          bool live_next = false;
          u64 c_next = fetch(t0, f_next, live_next);
          for (int64_t t = t0; t < t1; ++t) {
            const u64 c = c_next;
            const bool live = live_next;
            f = f_next;
            c_next = fetch(t + 1, f_next, live_next);
            const int n = (int)s_flagged[f];
            const u32 key = (u32)(c >> 32);
            const int s = (live && a.n_seg > 1) ? seg_of(composite_idx(c)) : 0;
            const u32 bound = live ? bound_of(f, n, s) : kFull;
            const bool use = bound != kFull && (bound >> 31) && key >= (bound & 0x7FFFFFFFu);
            u32* target = a.dhist + ((size_t)n * a.n_seg + s) * kBins + (key >> 19);
            const u32 act = __ballot_sync(kFull, use);
            if (use) {
              const u32 peers = __match_any_sync(act, (u64)(uintptr_t)target);
              if (lane == __ffs(peers) - 1) atomicAdd(target, (u32)__popc(peers));
            }
          }
        }
        if (p.use_marks) {  // the previous support: scores from the override list (index order)
          const int64_t per_w = (p.k + 31) / 32, tasks = nf * per_w;
          const int64_t per = (tasks + nwarps - 1) / nwarps;
          const int64_t t0 = gw * per, t1 = t0 + per < tasks ? t0 + per : tasks;
          for (int64_t t = t0; t < t1; ++t) {
            const int64_t f = t / per_w;
            const int n = (int)s_flagged[f];
            const int64_t i = (t - f * per_w) * 32 + lane;
            const bool live = i < p.k;
            const int32_t j = live ? p.prev_idx[(size_t)n * p.k + i] : 0;
            const u32 key = live ? __ldcg(&p.ovr_key[(size_t)n * p.k + i]) : 0u;
            const int s = (live && a.n_seg > 1) ? seg_of((u32)j) : 0;
            const u32 bound = live ? bound_of(f, n, s) : kFull;
            const bool part = bound != kFull;
            const u32 lo_seg = bound & 0x7FFFFFFFu;
            const bool use = part && key >= lo_seg;
            u32* hist = a.dhist + ((size_t)n * a.n_seg + s) * kBins;
            u32* target = hist + (key >> 19);
            const u32 act = __ballot_sync(kFull, use);
            if (use) {  // lanes that count into the same bin add once
              const u32 peers = __match_any_sync(act, (u64)(uintptr_t)target);
              if (lane == __ffs(peers) - 1) atomicAdd(target, (u32)__popc(peers));
            }
            // a segment counted from the rows has the entry under bits(|a|): take that back (a list-fed one never
            // counted it: the list has no entries of the previous support)
            if (part && !(bound >> 31)) {
              const u32 ka = __float_as_uint(p.eps[(size_t)n * p.ld + j]) & 0x7FFFFFFFu;
              if (ka >= lo_seg) atomicSub(hist + (ka >> 19), 1u);
            }
          }
        }
      } else
      if (lv == 0 && p.use_marks) {
        // the entries of the previous support, which the walk above left out: their scores come from the override
        // list (index order), one lane per entry, straight into the segments' histograms in global memory
        for (int64_t f = 0; f < nf; ++f) {
          const int n = (int)s_flagged[f];
          const int32_t* pi = p.prev_idx + (size_t)n * p.k;
          const u32* okey = p.ovr_key + (size_t)n * p.k;
          for (int64_t i0 = (int64_t)blockIdx.x * blockDim.x + (tid & ~31); i0 < p.k; i0 += (int64_t)gridDim.x * blockDim.x) {
            const int64_t i = i0 + lane;
            bool use = i < p.k;
            const int32_t j = use ? pi[i] : 0;
            const u32 key = use ? __ldcg(&okey[i]) : 0u;
            const int s = a.n_seg > 1 ? dense_seg_of_index(a.seg_end, a.n_seg, j) : 0;
            bool take_back = false;
            u32 lo_seg = 0;
            if (use) {
              const SegState st = load_seg(a, n, s);
              take_back = st.mode == want_mode && !(LAYERED && st.src);  // (a list-fed segment never counted it: the list has no such entries)
              lo_seg = st.lo;
              use = st.mode == want_mode && key >= st.lo;
            }
            u32* hist = a.dhist + ((size_t)n * a.n_seg + s) * kBins;
            u32* target = hist + (key >> 19);
            const u32 act = __ballot_sync(kFull, use);
            if (use) {  // lanes that count into the same bin add once
              const u32 peers = __match_any_sync(act, (u64)(uintptr_t)target);
              if (lane == __ffs(peers) - 1) atomicAdd(target, (u32)__popc(peers));
            }
            // the walk counted the entry under bits(|a|): take that back (the sums are what matters: a bin may
            // pass through "negative" values on the way)
            if (take_back) {
              const u32 ka = __float_as_uint(p.eps[(size_t)n * p.ld + j]) & 0x7FFFFFFFu;
              if (ka >= lo_seg) atomicSub(hist + (ka >> 19), 1u);
            }
          }
        }
      }
    };

    // Per segment that takes part: load its histogram (clearing it for the next use) and find the bin of the
    // need-th largest.  done(st, b, above, in_bin) runs in thread 0 and updates the state; b == kFull: the
    // histogram holds fewer than `need` entries.
    auto find_pass = [&](int lv, u32 want_mode, auto done) {
      for (int64_t v = blockIdx.x; v < nsegs; v += gridDim.x) {
        const int n = (int)s_flagged[v / a.n_seg], s = (int)(v % a.n_seg);
        const SegState old = load_seg(a, n, s);
        if (old.mode != want_mode) continue;  // the same in every thread of the block
        u32* gh = a.dhist + ((size_t)n * a.n_seg + s) * kBins;
        __syncthreads();
        for (int i = tid; i < kBins; i += blockDim.x) {
          s_hist[i] = __ldcg(&gh[i]);
          gh[i] = 0;  // ready for the next digit, and for the next launch
        }
        const u32 need = lv ? old.need : (u32)(a.seg_kpre[s + 1] - a.seg_kpre[s]);
        __syncthreads();
        block_find_from_top(s_hist, kBins, need, s_scan, s_res);
        const u32 b = s_res[0], above = s_res[1];
        // for the next round's bound: the bin of the entry three times as far down (first digit); in layer-wise mode,
        // after the second digit, the sub-bin of the entry max(k_s, 32) places below the threshold
        u32 b_wide = kFull;
        const u32 ks_seg = (u32)(a.seg_kpre[s + 1] - a.seg_kpre[s]);
        const u32 r2 = lv == 0 ? 3u * need : ((LAYERED && lv == 1) ? need + (ks_seg > 32u ? ks_seg : 32u) : 0u);
        if (r2 > need && b != kFull) {
          __syncthreads();
          block_find_from_top(s_hist, kBins, r2, s_scan, s_res);
          b_wide = s_res[0];
        }
        if (tid == 0) done(n, s, old, need, b, above, b == kFull ? 0u : s_hist[b], b_wide);
        __syncthreads();
      }
    };

    // The first digit's search, a warp per segment: the histogram is read (and cleared) from the top in runs of 512
    // bins, 16 per lane with lane 0 at the top, down to the run that holds the segment's lower bound (nothing was
    // counted below it).  It yields the bin b of the need-th largest entry, the entries above it and inside it, and
    // the bin of the entry three times as far down (next round's bound).  The worker's list space is dealt out by
    // the warp that finishes the worker's last segment, in segment order: a segment whose bin does not fit stays on
    // the rows and takes nothing from those after it.
    auto find_first = [&](int attempt) {
      const int64_t nwarps = (int64_t)gridDim.x * kDenseWarps;
      for (int64_t v = (int64_t)warp * gridDim.x + blockIdx.x; v < nsegs; v += nwarps) {  // (warps numbered across the blocks)
        const int n = (int)s_flagged[v / a.n_seg], s = (int)(v % a.n_seg);
        const SegState old = load_seg(a, n, s);
        SegState* st = a.seg + (size_t)n * a.n_seg + s;
        if (old.mode == kSegRetry) {  // the same in every lane
          const u32 need = (u32)(a.seg_kpre[s + 1] - a.seg_kpre[s]);
          uint4* gh = reinterpret_cast<uint4*>(a.dhist + ((size_t)n * a.n_seg + s) * kBins);
          const int run_lo = (int)(old.lo >> 19) >> 9;
          u32 cum = 0, b = kFull, above = 0, in_bin = 0, b_wide = kFull;
          uint4 nx[4];
#pragma unroll
          for (int i = 0; i < 4; ++i) nx[i] = __ldcg(gh + (kBins / 4 - 128) + (31 - lane) * 4 + i);
          for (int run = kBins / 512 - 1; run >= run_lo; --run) {
            uint4* g = gh + run * 128 + (31 - lane) * 4;  // this lane's 16 bins of the run
            u32 h[16] = {nx[0].x, nx[0].y, nx[0].z, nx[0].w, nx[1].x, nx[1].y, nx[1].z, nx[1].w,
                         nx[2].x, nx[2].y, nx[2].z, nx[2].w, nx[3].x, nx[3].y, nx[3].z, nx[3].w};
            if (run > run_lo) {
#pragma unroll
              for (int i = 0; i < 4; ++i) nx[i] = __ldcg(g - 128 + i);
            }
            u32 sum = 0;
#pragma unroll
            for (int i = 0; i < 16; ++i) sum += h[i];
            if (sum) {  // ready for the next digit, and for the next launch
#pragma unroll
              for (int i = 0; i < 4; ++i) g[i] = make_uint4(0u, 0u, 0u, 0u);
            }
            u32 incl = sum;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
              const u32 t = __shfl_up_sync(kFull, incl, o);
              if (lane >= o) incl += t;
            }
            const u32 before = cum + incl - sum;  // entries in higher bins than this lane's
#pragma unroll
            for (int pass = 0; pass < 2; ++pass) {
              const bool open = pass == 0 ? b == kFull : (b_wide == kFull && need <= kFull / 3u);
              const u32 r = pass == 0 ? need : 3u * need;
              const u32 hit = __ballot_sync(kFull, open && before < r && r <= before + sum);
              if (hit) {
                const int src = __ffs(hit) - 1;
                u32 fb = 0, fa = 0, fi = 0;
                if (lane == src) {
                  u32 acc = before;
#pragma unroll
                  for (int i = 15; i >= 0; --i) {
                    if (acc < r && r <= acc + h[i]) { fb = (u32)(run * 512 + (31 - lane) * 16 + i); fa = acc; fi = h[i]; }
                    acc += h[i];
                  }
                }
                fb = __shfl_sync(kFull, fb, src);
                if (pass == 0) {
                  b = fb;
                  above = __shfl_sync(kFull, fa, src);
                  in_bin = __shfl_sync(kFull, fi, src);
                } else {
                  b_wide = fb;
                }
              }
            }
            cum += __shfl_sync(kFull, incl, 31);
          }
          if (lane == 0 && !old.src && old.lo == 0u && !old.nonzero) {
            // the walk looked at every entry and saw no key but zero (scores on the previous support are zero where
            // the accumulator is): the segment's lowest k_s indices win; nothing to search, no list, no bound
            st->mode = kSegZero; st->prefix = 0; st->need = need; st->ties = 0;
            // layer-wise mode: the bound 1 for the next round: the streaming pass then gathers every entry of the layer
            // that is not zero, and a layer that sends none is known to be all zero without a walk
            a.seg_thr[(size_t)n * a.n_seg + s] = LAYERED ? 1u : 0u;
          } else if (lane == 0 && LAYERED && old.src && old.lo == 1u && cum == 0u) {
            // the bound was 1 and the candidate list holds no entry of this segment (nor has the override list one
            // with a score other than zero): every key is zero again
            st->mode = kSegZero; st->prefix = 0; st->need = need; st->ties = 0;
            a.seg_thr[(size_t)n * a.n_seg + s] = 1u;
          } else if (lane == 0) {
            if (b == kFull) {
              if (old.lo == 0u) {  // fewer than k entries in the whole segment: cannot happen
                atomicOr(&p.gctl->dense_flags, kFlagBad);
                st->mode = kSegList; st->prefix = 0; st->need = 0; st->ties = 0;
              } else {  // stays kSegRetry: first an octave lower, then without a bound; from the rows in any case
                st->src = 0u;
                st->lo = (attempt == 0 && old.lo > kOctave) ? old.lo - kOctave : 0u;
                atomicOr(&p.gctl->dense_flags, kFlagRetry | kFlagWalk);
              }
            } else {
              st->prefix = b;
              st->need = need - above;
              st->ties = in_bin;
              st->mode = kSegWant;
              // next round's lower bound: the lower edge of the bin that holds this round's 3k-th largest entry (but
              // at least one whole bin below the threshold's own: the bins are 1/16 octave wide); if fewer than that
              // were counted, two bins below this round's bound
              const u32 below = b > 0u ? b - 1u : 0u;
              u32 next;
              if (b_wide != kFull) {  // (enough entries were counted at or above this round's bound: no need to go below it)
                next = (b_wide < below ? b_wide : below) << 19;
                if (LAYERED && next < old.lo) next = old.lo;
              } else if (LAYERED) {   // a list segment whose bound lies inside the threshold's bin widens it itself
                const u32 gap = (b << 19) > old.lo ? ((b << 19) - old.lo) >> 1 : 0u;
                const u32 step = gap > 256u ? gap : 256u;
                next = (b << 19) > old.lo ? (old.lo > step ? old.lo - step : 0u) : old.lo;
              } else {
                next = old.lo > kHintMargin ? old.lo - kHintMargin : 0u;
              }
              a.seg_thr[(size_t)n * a.n_seg + s] = next & ~1u;
            }
          }
        }
        // the worker's last segment to be done deals out the list space
        u32 done = 0;
        __syncwarp();
        if (lane == 0) {
          __threadfence();
          done = atomicAdd(&p.ctl[n].seg_done, 1u);
        }
        done = __shfl_sync(kFull, done, 0);
        if (done + 1u != (u32)a.n_seg) continue;
        __threadfence();
        u32 fill = __ldcg(&p.ctl[n].bcount);
        for (int s0 = 0; s0 < a.n_seg; s0 += 32) {
          const int sx = s0 + lane;
          SegState* sp = a.seg + (size_t)n * a.n_seg + sx;
          const bool want = sx < a.n_seg && __ldcg(&sp->mode) == kSegWant;
          const u32 len = want ? __ldcg(&sp->ties) : 0u;
          u32 incl = len;
#pragma unroll
          for (int o = 1; o < 32; o <<= 1) {
            const u32 t = __shfl_up_sync(kFull, incl, o);
            if (lane >= o) incl = (incl + t < incl) ? kFull : incl + t;  // saturating
          }
          const u32 all = __shfl_sync(kFull, incl, 31);
          if (all != kFull && (u64)fill + all <= (u64)p.stride) {  // the usual case: all of them fit
            if (want) { sp->boff = fill + incl - len; sp->mode = kSegList; }
            fill += all;
          } else {  // one after the other
            for (int l = 0; l < 32; ++l) {
              const u32 ln = __shfl_sync(kFull, len, l);
              const bool wl = __shfl_sync(kFull, want ? 1u : 0u, l) != 0u;
              if (!wl) continue;
              const bool fits = (u64)fill + ln <= (u64)p.stride;
              if (lane == l) {
                if (fits) { sp->boff = fill; sp->mode = kSegList; }
                else { sp->mode = kSegRows; atomicOr(&p.gctl->dense_flags, kFlagRows); }
              }
              if (fits) fill += ln;
            }
          }
        }
        if (lane == 0) {
          p.ctl[n].bcount = fill;
          p.ctl[n].seg_done = 0u;
        }
      }
    };

    // ---- set-up: the lower bound each segment starts with ----
    for (int64_t v = (int64_t)blockIdx.x * blockDim.x + tid; v < nsegs; v += (int64_t)gridDim.x * blockDim.x) {
      const int n = (int)s_flagged[v / a.n_seg], s = (int)(v % a.n_seg);
      u32 lo;
      if (LAYERED) {
        lo = a.seg_thr[(size_t)n * a.n_seg + s];  // left by the last round (0: none)
      } else {
        // the sampled cutoff as it is when the path was asked for; an octave lower when that cutoff has just left
        // too few entries above it
        const u32 hint = p.ctl[n].hint;
        lo = hint == kFull ? 0u : (p.ctl[n].force_dense ? hint : (hint > kOctave ? hint - kOctave : 0u));
      }
      SegState st;
      st.prefix = 0; st.need = 0; st.ties = 0; st.mode = kSegRetry; st.lo = lo; st.boff = 0; st.bfill = 0; st.sh = 19;
      // layer-wise: the candidate list holds every entry of the segment at or above lo, unless there was no bound to
      // gather by or the list overflowed
      st.src = (LAYERED && lo != 0u && (u64)p.ctl[n].cand_count <= (u64)p.capA) ? 1u : 0u;
      if (LAYERED && !st.src) atomicOr(&p.gctl->dense_flags, kFlagWalk);
      st.nonzero = 0u;
      st.pad[0] = st.pad[1] = 0u;
      a.seg[(size_t)n * a.n_seg + s] = st;
    }
    grid.sync();

    // ---- (A) first digit; again with lo an octave lower, then with lo = 0, for the segments whose hint was too high ----
    for (int attempt = 0; attempt < 3; ++attempt) {
      hist_pass(0, kSegRetry, !LAYERED || (__ldcg(&p.gctl->dense_flags) & kFlagWalk));
      grid.sync();
      find_first(attempt);
      grid.sync();
      if (!(__ldcg(&p.gctl->dense_flags) & kFlagRetry)) break;  // the same in every block
      grid.sync();  // everyone has seen the flag
      if (blockIdx.x == 0 && tid == 0) atomicAnd(&p.gctl->dense_flags, ~kFlagRetry);
    }

    // ---- (B) second pass over the rows: winners above the bin, and the bin's own entries to their list ----
    auto compact_pass = [&](u32 want_mode, bool walk) {
      int cur_n = -1, cur_s = -1;
      // During the walk a thread that holds an entry at or above the bin's lower edge puts it into its warp's
      // staging list itself (one shared-memory counter).  When the list is half full, or the segment changes, the
      // warp writes it out: entries on the previous support are dropped (their scores come from the override list),
      // entries above the bin win (mask bit, winner list), the bin's own go to the segment's in-bin list.
      u64* list = listA;  // both halves of the warp's staging space: 2 * kWarpList entries
      constexpr u32 kCap = 2u * kWarpList;
      auto marked = [&](int n, u32 j) {
        return p.use_marks && ((__ldg(p.mask_old + (size_t)n * p.W + (j >> 5)) >> (j & 31)) & 1u);
      };
      auto place = [&](int n, int s, const SegState& sg, u64 c, bool live) {  // all lanes of the warp; live: this lane has an entry
        const bool isA = live && (u32)(c >> (32u + sg.sh)) > sg.prefix;  // the key's digits fixed so far
        const bool isB = live && !isA;
        const u32 mA = __ballot_sync(kFull, isA), mB = __ballot_sync(kFull, isB);
        u32 baseA = 0, baseB = 0;
        if (lane == 0 && mA) baseA = atomicAdd(&p.ctl[n].acount, (u32)__popc(mA));
        if (lane == 0 && mB) baseB = atomicAdd(&a.seg[(size_t)n * a.n_seg + s].bfill, (u32)__popc(mB));
        baseA = __shfl_sync(kFull, baseA, 0);
        baseB = __shfl_sync(kFull, baseB, 0);
        const u32 lt = (1u << lane) - 1u;
        if (isA) {
          set_winner(p.mask_new + (size_t)n * p.W, composite_idx(c), p.d);
          const u32 pos = baseA + __popc(mA & lt);
          if (RT_INB(pos < k)) p.ovr_comp[(size_t)n * p.k + pos] = c;
        }
        if (isB) {
          const u32 pos = baseB + __popc(mB & lt);
          if (RT_INB(pos < sg.ties)) p.candB[(size_t)n * p.stride + sg.boff + pos] = c;
        }
      };
      auto flush = [&](int n, int s, const SegState& sg) {  // every lane of the warp
        __syncwarp();
        u32 c = *reinterpret_cast<volatile u32*>(&s_wcnt[0][warp]);
        c = c < kCap ? c : kCap;
        if (p.use_marks && c) c = warp_drop_marked(list, c, p.mask_old + (size_t)n * p.W, lane);
        for (u32 i0 = 0; i0 < c; i0 += 32) place(n, s, sg, i0 + lane < c ? list[i0 + lane] : 0ull, i0 + lane < c);
        __syncwarp();
        if (lane == 0) s_wcnt[0][warp] = 0;
        __syncwarp();
      };
      // A region dense with winners can fill the list within one step of the walk; an entry that finds it full
      // goes out by itself.
      auto direct = [&](int n, int s, const SegState& sg, u64 c) {
        const u32 j = composite_idx(c);
        if (marked(n, j)) return;
        if ((u32)(c >> (32u + sg.sh)) > sg.prefix) {
          set_winner(p.mask_new + (size_t)n * p.W, j, p.d);
          const u32 pos = atomicAdd(&p.ctl[n].acount, 1u);
          if (RT_INB(pos < k)) p.ovr_comp[(size_t)n * p.k + pos] = c;
        } else {
          const u32 pos = atomicAdd(&a.seg[(size_t)n * a.n_seg + s].bfill, 1u);
          if (RT_INB(pos < sg.ties)) p.candB[(size_t)n * p.stride + sg.boff + pos] = c;
        }
      };
      if (lane == 0) s_wcnt[0][warp] = 0;
      __syncwarp();
      SegState st;
      st.mode = ~0u;
      for (int64_t c0 = walk ? (int64_t)blockIdx.x * t_run : total_tiles; c0 < total_tiles; c0 += t_step)
      for (int64_t w = c0, c1 = c0 + t_run < total_tiles ? c0 + t_run : total_tiles; w < c1; ++w) {
        const DenseTile t = dense_tile(a, s_flagged, w);
        if (t.n != cur_n || t.s != cur_s) {
          if (cur_n >= 0 && st.mode == want_mode) flush(cur_n, cur_s, st);
          cur_n = t.n; cur_s = t.s;
          st = load_seg(a, t.n, t.s);  // but for its fill counter, nothing writes it during this pass
        }
        if (st.mode != want_mode || (LAYERED && want_mode == kSegList && st.src)) { w += a.seg_tile0[t.s + 1] - 1 - t.t; continue; }  // nothing to do in this segment: on to its last tile (the same in every thread of the block)
        const u32 floor_key = max(st.prefix << st.sh, st.lo);  // nothing below it is a winner or in the bin
        dense_walk<true, true>(p, t.n, t.t0, t.t1, floor_key,
          [&](int64_t j4, const u32 (&key)[4], const bool (&in)[4]) {
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              if (!in[q] || key[q] < floor_key) continue;
              const u64 c = make_composite(key[q], (u32)(j4 + q));
              const u32 at = atomicAdd(&s_wcnt[0][warp], 1u);
              if (at < kCap) list[at] = c;
              else direct(t.n, t.s, st, c);
            }
          },
          [&]() {
            if (*reinterpret_cast<volatile u32*>(&s_wcnt[0][warp]) >= kCap / 2u) flush(t.n, t.s, st);
          });
      }
      if (cur_n >= 0 && st.mode == want_mode) flush(cur_n, cur_s, st);
      u32 cntA = 0;  // from here on the lists are filled by ballot: warp-uniform fill
      if (LAYERED && want_mode == kSegList) {
        // Layer-wise mode: the candidate lists of the segments fed from them, then the override list, as runs of
        // 32-entry tasks over all flagged workers, dealt to the warps of the grid in contiguous pieces (as in the
        // histogram pass).  Each warp keeps the first half of its staging space for the winners it finds; the
        // other halves hold, when they fit, what is needed of every segment's state.
        __syncthreads();  // every warp has written out what the walk above staged
        u64* listL = s_stage + (size_t)warp * kWarpList;
        uint4* t_seg = reinterpret_cast<uint4*>(s_stage + (size_t)kDenseWarps * kWarpList);  // [nsegs]: prefix | flags, bound, list offset, list length
        u32* t_end = s_hist;                                                                // [n_seg]
        const bool fast = (u64)nsegs * 2u <= (u64)kDenseWarps * kWarpList && a.n_seg <= kBins;
        constexpr u32 kPart = 1u << 31, kFed = 1u << 30;
        auto pack = [&](const SegState& sg) {
          return make_uint4(sg.prefix | (sg.mode == kSegList ? kPart : 0u) | (sg.src ? kFed : 0u), sg.lo, sg.boff, sg.ties);
        };
        if (fast) {
          for (int i = tid; i < a.n_seg; i += blockDim.x) t_end[i] = (u32)a.seg_end[i];
          for (int64_t v = tid; v < nsegs; v += blockDim.x)
            t_seg[v] = pack(load_seg(a, (int)s_flagged[v / a.n_seg], (int)(v % a.n_seg)));
          __syncthreads();
        }
        auto seg_of = [&](u32 j) -> int {
          if (!fast) return dense_seg_of_index(a.seg_end, a.n_seg, (int64_t)j);
          int lo = 0, hi = a.n_seg - 1;  // the first segment whose end lies beyond j
          while (lo < hi) {
            const int mid = (lo + hi) >> 1;
            if (t_end[mid] <= j) lo = mid + 1; else hi = mid;
          }
          return lo;
        };
        auto info_of = [&](int64_t f, int n, int s) -> uint4 {
          return fast ? t_seg[f * a.n_seg + s] : pack(load_seg(a, n, s));
        };
        int cur = -1;  // the worker whose winners the warp is staging
        auto flush_L = [&]() {
          if (cur >= 0) stage_flush(listL, cntA, &p.ctl[cur].acount, p.ovr_comp + (size_t)cur * p.k, (u64)k, lane);
        };
        // one task's entries (c: composite, live: this lane has one; fed_only: candidates count for list-fed segments only)
        auto place_task = [&](int64_t f, int n, u64 c, bool live, bool fed_only) {
          if (n != cur) { flush_L(); cur = n; }
          const u32 key = (u32)(c >> 32), j = composite_idx(c);
          const int s = (live && a.n_seg > 1) ? seg_of(j) : 0;
          uint4 sg = make_uint4(0u, 0u, 0u, 0u);
          if (live) sg = info_of(f, n, s);
          const bool part = (sg.x & kPart) && (!fed_only || (sg.x & kFed));
          const u32 prefix = sg.x & 0x00FFFFFFu;
          const bool win = part && (key >> 19) > prefix;
          const bool bin = part && (key >> 19) == prefix && key >= sg.y;
          if (win) set_winner(p.mask_new + (size_t)n * p.W, j, p.d);
          const u32 act = __ballot_sync(kFull, bin);
          if (bin) {  // the bin's entries to their segment's list: lanes of one segment reserve their places together
            const u32 peers = __match_any_sync(act, (u32)s);
            const int leader = __ffs(peers) - 1;
            u32 base = 0;
            if (lane == leader) base = atomicAdd(&a.seg[(size_t)n * a.n_seg + s].bfill, (u32)__popc(peers));
            base = __shfl_sync(peers, base, leader);
            const u32 pos = base + (u32)__popc(peers & ((1u << lane) - 1u));
            if (RT_INB(pos < sg.w)) p.candB[(size_t)n * p.stride + sg.z + pos] = c;
          }
          if (__any_sync(kFull, win)) {
            stage_add(listL, cntA, win, c, lane);
            if (cntA >= (u32)(kWarpList - 32)) flush_L();
          }
        };
        const int64_t gw = (int64_t)warp * gridDim.x + blockIdx.x, nwarps = (int64_t)gridDim.x * kDenseWarps;  // warps numbered across the blocks: a short run of tasks spreads over all SMs
        {  // candidates
          const int64_t tasks = s_cbase[nf];
          const int64_t per = (tasks + nwarps - 1) / nwarps;
          const int64_t t0 = gw * per, t1 = t0 + per < tasks ? t0 + per : tasks;
          int64_t f = 0;
          if (t0 < t1) {
            int64_t lo = 0, hi = nf;  // the worker whose tasks include t0
            while (hi - lo > 1) {
              const int64_t mid = (lo + hi) >> 1;
              if ((int64_t)s_cbase[mid] <= t0) lo = mid; else hi = mid;
            }
            f = lo;
          }
          auto fetch = [&](int64_t t, int64_t& ff, bool& live) -> u64 {
            live = false;
            if (t >= t1) return 0ull;
            while (t >= (int64_t)s_cbase[ff + 1]) ++ff;
            const int n = (int)s_flagged[ff];
            const int64_t i = (t - (int64_t)s_cbase[ff]) * 32 + lane;
            live = i < (int64_t)p.ctl[n].cand_count;
            return live ? __ldcg(p.candA + (size_t)n * p.stride + i) : 0ull;
          };
          int64_t f_next = f;
          bool live_next = false;
          u64 c_next = fetch(t0, f_next, live_next);
          for (int64_t t = t0; t < t1; ++t) {
            const u64 c = c_next;
            const bool live = live_next;
            f = f_next;
            c_next = fetch(t + 1, f_next, live_next);
            place_task(f, (int)s_flagged[f], c, live, true);
          }
        }
        if (p.use_marks) {  // the previous support: scores from the override list
          const int64_t per_w = (p.k + 31) / 32, tasks = nf * per_w;
          const int64_t per = (tasks + nwarps - 1) / nwarps;
          const int64_t t0 = gw * per, t1 = t0 + per < tasks ? t0 + per : tasks;
          for (int64_t t = t0; t < t1; ++t) {
            const int64_t f = t / per_w;
            const int n = (int)s_flagged[f];
            const int64_t i = (t - f * per_w) * 32 + lane;
            const bool live = i < p.k;
            const int32_t j = live ? p.prev_idx[(size_t)n * p.k + i] : 0;
            const u32 key = live ? __ldcg(&p.ovr_key[(size_t)n * p.k + i]) : 0u;
            place_task(f, n, make_composite(key, (u32)j), live, false);
          }
        }
        flush_L();
        __syncthreads();  // the tables in shared memory are free again: a histogram pass may follow at once
        return;
      }
      auto flush_A2 = [&](int n) {
        stage_flush(listA, cntA, &p.ctl[n].acount, p.ovr_comp + (size_t)n * p.k, (u64)k, lane);
      };
      if (p.use_marks) {  // the same for the entries of the previous support, from the override list
        for (int64_t f = 0; f < nf; ++f) {
          const int n = (int)s_flagged[f];
          const int32_t* pi = p.prev_idx + (size_t)n * p.k;
          const u32* okey = p.ovr_key + (size_t)n * p.k;
          u32* mask = p.mask_new + (size_t)n * p.W;
          for (int64_t i0 = (int64_t)blockIdx.x * blockDim.x + (tid & ~31); i0 < p.k; i0 += (int64_t)gridDim.x * blockDim.x) {
            const int64_t i = i0 + lane;
            const bool live = i < p.k;
            const int32_t j = live ? pi[i] : 0;
            const u32 key = live ? __ldcg(&okey[i]) : 0u;
            const int s = a.n_seg > 1 ? dense_seg_of_index(a.seg_end, a.n_seg, j) : 0;
            bool win = false, bin = false;
            SegState st;
            st.boff = 0; st.ties = 0;
            if (live) {
              st = load_seg(a, n, s);
              if (st.mode == want_mode) {
                win = (key >> st.sh) > st.prefix;
                bin = (key >> st.sh) == st.prefix && key >= st.lo;
              }
            }
            const u64 c = make_composite(key, (u32)j);
            if (win) set_winner(mask, (u32)j, p.d);
            {  // the bin's entries to their segment's list: lanes of one segment reserve their places together
              const u32 act = __ballot_sync(kFull, bin);
              if (bin) {
                const u32 peers = __match_any_sync(act, (u32)s);
                const int leader = __ffs(peers) - 1;
                u32 base = 0;
                if (lane == leader) base = atomicAdd(&a.seg[(size_t)n * a.n_seg + s].bfill, (u32)__popc(peers));
                base = __shfl_sync(peers, base, leader);
                const u32 pos = base + (u32)__popc(peers & ((1u << lane) - 1u));
                if (RT_INB(pos < st.ties)) p.candB[(size_t)n * p.stride + st.boff + pos] = c;
              }
            }
            if (__any_sync(kFull, win)) {
              stage_add(listA, cntA, win, c, lane);
              if (cntA >= (u32)(kWarpList - 32)) flush_A2(n);
            }
          }
          flush_A2(n);
        }
      }
    };
    const u32 flags0 = __ldcg(&p.gctl->dense_flags);  // written before the last barrier
    compact_pass(kSegList, !LAYERED || (flags0 & kFlagWalk));
    if (flags0 & kFlagRows) hist_pass(1, kSegRows, true);
    grid.sync();

    // ---- (C) per list segment: the `need` largest composites of its in-bin list win ----
    // Layer-wise mode: the lower bound a list segment leaves for the next round.  Error feedback packs more and more
    // entries right under the threshold, so the bound goes by rank, not by magnitude: it is the key of the entry
    // max(k_s, 32) places below the threshold in the segment's in-bin list (bound_rank: its place in that list).
    // A list too short for that (few entries at or above this round's bound) widens the gap between the bound and
    // the threshold key by a half, as long as the bound lies inside the threshold's bin; otherwise the bin edge that
    // the first digit's search left stands.
    auto bound_rank = [&](const SegState& sg, int s) -> u32 {
      const u32 ks = (u32)(a.seg_kpre[s + 1] - a.seg_kpre[s]);
      const u32 more = ks > 32u ? (ks > kFull / 4u ? kFull / 2u : ks) : 32u;
      return sg.need + more < more ? kFull : sg.need + more;
    };
    auto leave_rank_bound = [&](int n, int s, const SegState& sg, u32 key_r) {  // one thread
      if (!LAYERED || sg.mode != kSegList) return;
      a.seg_thr[(size_t)n * a.n_seg + s] = key_r & ~1u;
    };
    auto leave_wider_bound = [&](int n, int s, const SegState& sg, u32 t_key) {  // one thread
      if (!LAYERED || sg.mode != kSegList) return;
      const u32 edge = sg.prefix << 19;
      if (sg.lo <= edge) return;
      const u32 gap = t_key > sg.lo ? (t_key - sg.lo) >> 1 : 0u;
      const u32 step = gap > 256u ? gap : 256u;
      a.seg_thr[(size_t)n * a.n_seg + s] = (sg.lo - edge > step ? sg.lo - step : edge) & ~1u;
    };
    auto list_select = [&](u32 want_mode) {
     for (int64_t v = blockIdx.x; v < nsegs; v += gridDim.x) {
      const int n = (int)s_flagged[v / a.n_seg], s = (int)(v % a.n_seg);
      const SegState st = load_seg(a, n, s);
      u32* mask = p.mask_new + (size_t)n * p.W;
      if (want_mode == kSegList && st.mode == kSegZero) {  // an all-zero segment: its first k_s coordinates
        __syncthreads();
        if (tid == 0) s_cnt = atomicAdd(&p.ctl[n].acount, st.need);
        __syncthreads();
        const u32 first = (u32)(s ? a.seg_end[s - 1] : 0);
        for (u32 i = tid; i < st.need; i += blockDim.x) {
          set_winner(mask, first + i, p.d);
          if (RT_INB((u64)s_cnt + i < (u64)k)) p.ovr_comp[(size_t)n * p.k + s_cnt + i] = make_composite(0u, first + i);
        }
        __syncthreads();
        continue;
      }
      if (st.mode != want_mode || st.need == 0u) continue;  // the same in every thread of the block
      const u64* list = p.candB + (size_t)n * p.stride + st.boff;
      const u32 count = st.ties;
      if (st.bfill != count) {
        if (tid == 0) atomicOr(&p.gctl->dense_flags, kFlagBad);
        continue;
      }
      const u32 r_bound = LAYERED ? bound_rank(st, s) : kFull;  // place in the list of the entry whose key is the next bound
      if (count <= blockDim.x) {
        // a short list (the usual case): every thread ranks its entry against all others in shared memory; the
        // entry with `above` larger ones before it takes place `above` among the segment's winners from this list
        u64* items = reinterpret_cast<u64*>(s_hist);
        __syncthreads();
        const u64 mine = (u32)tid < count ? __ldcg(&list[tid]) : 0ull;
        if ((u32)tid < count) items[tid] = mine;
        if (tid == 0) s_cnt = atomicAdd(&p.ctl[n].acount, st.need);
        __syncthreads();
        if ((u32)tid < count) {
          u32 above = 0;
          for (u32 j = 0; j < count; ++j) above += items[j] > mine ? 1u : 0u;
          if (count >= r_bound ? above + 1u == r_bound : above + 1u == st.need) {
            if (count >= r_bound) leave_rank_bound(n, s, st, (u32)(mine >> 32));
            else leave_wider_bound(n, s, st, (u32)(mine >> 32));
          }
          if (above < st.need) {
            set_winner(mask, composite_idx(mine), p.d);
            if (RT_INB((u64)s_cnt + above < (u64)k)) p.ovr_comp[(size_t)n * p.k + s_cnt + above] = mine;
          }
        }
        __syncthreads();
        continue;
      }
      // A longer list: the need-th largest composite T, digit by digit: the key bits below the digits already fixed
      // first (19 as 11 + 8, or 7), then, only while entries of one key are still to be told apart, the index
      // bytes.  A digit whose bin is taken whole ends the search: the bin's lower edge is T.  The entries that are
      // still in play sit in shared memory (the warps' staging space, free in this phase): the whole list if it
      // fits, otherwise what the first digits leave of it, gathered in the pass that also emits the entries above.
      u64* items = s_stage;
      constexpr u32 kItems = (u32)(kDenseWarps * 2 * kWarpList);
      u64* A = p.ovr_comp + (size_t)n * p.k;
      __syncthreads();
      if (tid == 0) {
        s_res[0] = atomicAdd(&p.ctl[n].acount, st.need);  // the segment's places in the worker's winner list
        s_cnt = 0;                                        // winners placed so far
        s_nf2 = 0;                                        // entries gathered in shared memory
      }
      __syncthreads();
      const u32 abase = s_res[0];
      auto emit = [&](bool won, u64 c) {  // every lane of the warp
        const u32 mw = __ballot_sync(kFull, won);
        if (!mw) return;
        u32 at = 0;
        if (lane == 0) at = atomicAdd(&s_cnt, (u32)__popc(mw));
        at = __shfl_sync(kFull, at, 0) + (u32)__popc(mw & ((1u << lane) - 1u));
        if (won) {
          set_winner(mask, composite_idx(c), p.d);
          if (RT_INB(at < st.need && (u64)abase + at < (u64)k)) A[(u64)abase + at] = c;
        }
      };
      const u32 rounded = (count + 31u) & ~31u;
      if (st.need >= count) {  // all of them
        for (u32 i = tid; i < rounded; i += blockDim.x) emit(i < count, i < count ? __ldcg(&list[i]) : 0ull);
        __syncthreads();
        continue;
      }
      bool in_smem = count <= kItems;
      u32 m = count;  // entries in play
      if (in_smem) {
        for (u32 i0 = tid; i0 < count; i0 += 4u * blockDim.x) {  // four loads in flight
          u64 v[4];
#pragma unroll
          for (int q = 0; q < 4; ++q) v[q] = i0 + q * blockDim.x < count ? __ldcg(&list[i0 + q * blockDim.x]) : 0ull;
#pragma unroll
          for (int q = 0; q < 4; ++q)
            if (i0 + q * blockDim.x < count) items[i0 + q * blockDim.x] = v[q];
        }
      }
      u32 need = st.need;
      u64 prefix = (u64)st.prefix;  // every entry of the list has these digits
      int top = 32 + (int)st.sh;    // composite bits below the prefix
      bool bad = false, have_T = false;
      while (top > 0) {
        const int width = top > 32 ? (top - 32 > 11 ? 11 : top - 32) : 8;
        const int shift = top - width, bins = 1 << width;
        __syncthreads();
        for (int i = tid; i < bins; i += blockDim.x) s_hist[i] = 0;
        __syncthreads();
        if (in_smem) {
          for (u32 i = tid; i < m; i += blockDim.x) {
            const u64 c = items[i];
            if ((c >> top) == prefix) atomicAdd(&s_hist[(u32)(c >> shift) & (u32)(bins - 1)], 1u);
          }
        } else {
          for (u32 i0 = tid; i0 < m; i0 += 4u * blockDim.x) {  // four loads in flight
            u64 v[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) v[q] = i0 + q * blockDim.x < m ? __ldcg(&list[i0 + q * blockDim.x]) : 0ull;
#pragma unroll
            for (int q = 0; q < 4; ++q)
              if (i0 + q * blockDim.x < m && (v[q] >> top) == prefix)
                atomicAdd(&s_hist[(u32)(v[q] >> shift) & (u32)(bins - 1)], 1u);
          }
        }
        __syncthreads();
        block_find_from_top(s_hist, bins, need, s_scan, s_res + 1);
        const u32 bb = s_res[1], above = s_res[2];
        if (bb == kFull) { bad = true; break; }  // the same in every thread
        if (LAYERED && top == 32 + (int)st.sh && count >= r_bound && shift >= 32) {
          // (first digit: the histogram covers the whole list) the sub-bin of the entry that gives the next bound
          __syncthreads();  // everyone has read the first search's result
          block_find_from_top(s_hist, bins, r_bound, s_scan, s_res + 1);
          if (tid == 0 && s_res[1] != kFull)
            leave_rank_bound(n, s, st, (u32)((((prefix << width) | (u64)s_res[1]) << (shift - 32))));
          __syncthreads();
        }
        need -= above;
        prefix = (prefix << width) | (u64)bb;
        top = shift;
        const u32 in_bin = s_hist[bb];
        if (in_bin == need) break;  // all of this bin win
        if (in_bin <= blockDim.x) {
          // few entries are left in play: they are ranked against one another, and the need-th largest is T
          u64* ties = reinterpret_cast<u64*>(s_hist);
          __syncthreads();  // everyone has read the histogram
          if (tid == 0) s_nf2 = 0;
          __syncthreads();
          for (u32 i = tid; i < m; i += blockDim.x) {
            const u64 c = in_smem ? items[i] : __ldcg(&list[i]);
            if ((c >> top) == prefix) {
              const u32 at = atomicAdd(&s_nf2, 1u);
              if (RT_INB(at < blockDim.x)) ties[at] = c;
            }
          }
          __syncthreads();
          if (s_nf2 != in_bin) { bad = true; break; }  // the same in every thread
          if ((u32)tid < in_bin) {
            const u64 mine = ties[tid];
            u32 above = 0;
            for (u32 j = 0; j < in_bin; ++j) above += ties[j] > mine ? 1u : 0u;
            if (above + 1u == need) s_T = mine;
          }
          __syncthreads();
          have_T = true;
          break;
        }
        if (!in_smem && in_bin <= kItems) {
          // one pass over the list: what lies above the digits found so far wins now, what matches them moves to
          // shared memory and the search goes on there
          for (u32 i0 = tid; i0 < rounded; i0 += 4u * blockDim.x) {  // four loads in flight; whole warps take each step
            u64 v[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) v[q] = i0 + q * blockDim.x < count ? __ldcg(&list[i0 + q * blockDim.x]) : 0ull;
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              const u32 i = i0 + q * blockDim.x;
              if (i - lane >= rounded) break;  // the same in every lane
              const u64 c = v[q];
              const u64 hi = c >> top;
              emit(i < count && hi > prefix, c);
              const u32 mk = __ballot_sync(kFull, i < count && hi == prefix);
              if (mk) {
                u32 at = 0;
                if (lane == 0) at = atomicAdd(&s_nf2, (u32)__popc(mk));
                at = __shfl_sync(kFull, at, 0) + (u32)__popc(mk & ((1u << lane) - 1u));
                if (i < count && hi == prefix && RT_INB(at < kItems)) items[at] = c;
              }
            }
          }
          in_smem = true;
          m = in_bin;
        }
      }
      if (bad) {
        if (tid == 0) atomicOr(&p.gctl->dense_flags, kFlagBad);
        continue;
      }
      __syncthreads();
      const u64 T = have_T ? s_T : prefix << top;  // the lowest composite that wins
      if (tid == 0 && count < r_bound) leave_wider_bound(n, s, st, (u32)(T >> 32));
      const u32 mr = (m + 31u) & ~31u;
      for (u32 i = tid; i < mr; i += blockDim.x) {
        const u64 c = i < m ? (in_smem ? items[i] : __ldcg(&list[i])) : 0ull;
        emit(i < m && c >= T, c);
      }
      __syncthreads();
      if (tid == 0 && s_cnt != st.need) atomicOr(&p.gctl->dense_flags, kFlagBad);
     }
    };
    list_select(kSegList);
    if (flags0 & kFlagRows) {
      // Second digit of the segments whose first bin was too crowded for the list space.  After it the bin is 4096
      // times narrower: if it fits now, the segment goes the list way from here (one more pass over the rows);
      // otherwise (rows of equal keys) the third digit and the ordered take of ties follow.
      find_pass(1, kSegRows, [&](int n, int s, const SegState& old, u32 need, u32 b, u32 above, u32 in_bin, u32 b_rank) {
        SegState* st = a.seg + (size_t)n * a.n_seg + s;
        if (b == kFull) { atomicOr(&p.gctl->dense_flags, kFlagBad); b = 0; above = 0; }
        // (layer-wise mode) a bound by rank for the next round, as the list segments leave one: without it the bin edge
        // from the first digit stands, a sixteenth of an octave wide, and the next candidate list overflows
        if (LAYERED && b_rank != kFull) a.seg_thr[(size_t)n * a.n_seg + s] = (((old.prefix << 12) | b_rank) << 7) & ~1u;
        st->prefix = (old.prefix << 12) | b;
        st->need = need - above;
        st->ties = in_bin;
        st->sh = 7;
        u32 off;
        if (reserve_list_space(&p.ctl[n].bcount, in_bin, (u64)p.stride, &off)) {
          st->mode = kSegList2;
          st->boff = off;
          st->lo = 0u;  // the second digit counted every entry with the first digit's prefix
        } else {
          atomicOr(&p.gctl->dense_flags, kFlagRows2);
        }
      });
      grid.sync();
      const u32 flags_b = __ldcg(&p.gctl->dense_flags);
      compact_pass(kSegList2, true);
      if (flags_b & kFlagRows2) hist_pass(2, kSegRows, true);
      grid.sync();
      list_select(kSegList2);
     if (flags_b & kFlagRows2) {
      find_pass(2, kSegRows, [&](int n, int s, const SegState& old, u32 need, u32 b, u32 above, u32 in_bin, u32) {
        SegState* st = a.seg + (size_t)n * a.n_seg + s;
        if (b == kFull) { atomicOr(&p.gctl->dense_flags, kFlagBad); b = 0; above = 0; }
        st->prefix = (old.prefix << 7) | b;
        st->need = need - above;
        st->ties = in_bin;
        if (in_bin > need - above) atomicOr(&p.gctl->dense_flags, kFlagOrdered);
      });
      grid.sync();
      const u32 flags1 = __ldcg(&p.gctl->dense_flags);

      // ties in index order: per tile the number of entries equal to the threshold key T, then, per segment, the
      // number of them in lower tiles
      if (flags1 & kFlagOrdered) {
        for (int64_t w = w_begin; w < w_end; ++w) {
          const DenseTile t = dense_tile(a, s_flagged, w);
          const SegState st = load_seg(a, t.n, t.s);
          if (st.mode != kSegRows || st.ties <= st.need) { w += a.seg_tile0[t.s + 1] - 1 - t.t; continue; }  // nothing to do in this segment: on to its last tile (the same in every thread of the block)
          if (tid == 0) s_cnt = 0;
          __syncthreads();
          u32 mine = 0;
          dense_walk<false>(p, t.n, t.t0, t.t1, st.prefix, [&](int64_t, const u32 (&key)[4], const bool (&in)[4]) {
#pragma unroll
            for (int q = 0; q < 4; ++q) mine += (in[q] && key[q] == st.prefix) ? 1u : 0u;
          });
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) mine += __shfl_xor_sync(kFull, mine, o);
          if (lane == 0 && mine) atomicAdd(&s_cnt, mine);
          __syncthreads();
          if (tid == 0) a.tile_ties[2 * ((size_t)t.n * a.tiles + t.t)] = s_cnt;
          __syncthreads();
        }
        grid.sync();
        for (int64_t v = blockIdx.x; v < nsegs; v += gridDim.x) {
          const int n = (int)s_flagged[v / a.n_seg], s = (int)(v % a.n_seg);
          const SegState st = load_seg(a, n, s);
          if (st.mode != kSegRows || st.ties <= st.need) continue;  // the same in every thread of the block
          u32* tt = a.tile_ties + 2 * (size_t)n * a.tiles;
          u32 carry = 0;
          for (int64_t c0 = a.seg_tile0[s]; c0 < a.seg_tile0[s + 1]; c0 += blockDim.x) {
            const int64_t c = c0 + tid;
            const u32 mine = c < a.seg_tile0[s + 1] ? __ldcg(&tt[2 * c]) : 0u;
            u32 total;
            const u32 before = block_excl_scan(mine, s_scan, &total);
            if (c < a.seg_tile0[s + 1]) tt[2 * c + 1] = carry + before;
            carry += total;
          }
        }
        grid.sync();
      }
      // last pass over the rows of those segments: winners are the entries above T and the ties that are taken
      {
        u32 cntA = 0;
        int cur_n = -1;
        auto flush_A = [&](int n) {
          stage_flush(listA, cntA, &p.ctl[n].acount, p.ovr_comp + (size_t)n * p.k, (u64)k, lane);
        };
        for (int64_t w = w_begin; w < w_end; ++w) {
          const DenseTile t = dense_tile(a, s_flagged, w);
          if (t.n != cur_n) {
            if (cur_n >= 0) flush_A(cur_n);
            cur_n = t.n;
          }
          const SegState st = load_seg(a, t.n, t.s);
          if (st.mode != kSegRows) { w += a.seg_tile0[t.s + 1] - 1 - t.t; continue; }  // nothing to do in this segment: on to its last tile (the same in every thread of the block)
          const u32 T = st.prefix, need = st.need;
          // all of the tile's ties win, none of them, or (one tile per segment at most) the first few in index order
          bool all_win = st.ties <= need, none_win = false;
          u32 tie_rank = 0;
          if (!all_win) {
            const u32 here = __ldcg(&a.tile_ties[2 * ((size_t)t.n * a.tiles + t.t)]);
            tie_rank = __ldcg(&a.tile_ties[2 * ((size_t)t.n * a.tiles + t.t) + 1]);
            all_win = tie_rank + here <= need;
            none_win = tie_rank >= need;
          }
          const bool in_order = !all_win && !none_win;
          u32* mask = p.mask_new + (size_t)t.n * p.W;
          dense_walk<false>(p, t.n, t.t0, t.t1, in_order ? 0u : T, [&](int64_t j4, const u32 (&key)[4], const bool (&in)[4]) {
            bool win[4];
            u32 eq = 0;
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              win[q] = in[q] && (key[q] > T || (key[q] == T && all_win));
              eq += (in[q] && key[q] == T) ? 1u : 0u;
            }
            if (in_order) {  // the same in every thread of the block; threads hold consecutive quads
              u32 total;
              u32 r = tie_rank + block_excl_scan(eq, s_scan, &total);
#pragma unroll
              for (int q = 0; q < 4; ++q) {
                if (in[q] && key[q] == T) {
                  win[q] = r < need;
                  ++r;
                }
              }
              tie_rank += total;
            }
            u32 bits = 0;
#pragma unroll
            for (int q = 0; q < 4; ++q) bits |= win[q] ? (1u << q) : 0u;
            if (bits && RT_INB(j4 + 3 < p.W * 32)) atomicOr(&mask[j4 >> 5], bits << (j4 & 31));
            if (__any_sync(kFull, bits != 0u)) {
#pragma unroll
              for (int q = 0; q < 4; ++q) stage_add(listA, cntA, win[q], make_composite(key[q], (u32)(j4 + q)), lane);
              if (cntA >= (u32)(kWarpList - 128)) flush_A(t.n);
            }
          });
        }
        if (cur_n >= 0) flush_A(cur_n);
      }
     }
    }
    grid.sync();
    // every flagged worker must have gathered exactly k winners
    const u32 flags2 = __ldcg(&p.gctl->dense_flags);
    for (int64_t f = blockIdx.x; f < nf; f += gridDim.x) {
      if (tid == 0) {
        const int n = (int)s_flagged[f];
        if ((flags2 & kFlagBad) || __ldcg(&p.ctl[n].acount) != k) atomicOr(&p.gctl->err, kErrDenseSelect);
        p.ctl[n].took_dense = 1u;
      }
    }

    if (a.finish) {
      // ---- ranks and emission, as in k_post: per-quad prefix counts of the mask, segment bases, then every
      //      winner looks its rank up and writes its pair ----
      const int nw = blockDim.x >> 5;
      const int64_t U = p.W >> 3;
      const int64_t seg_units = (U + a.emit_segments - 1) / a.emit_segments;
      for (int64_t it = (int64_t)warp * gridDim.x + blockIdx.x; it < nf * a.emit_segments; it += (int64_t)gridDim.x * nw)  // (warps numbered across the blocks)
        post_prefix_segment(p, (int)s_flagged[it / a.emit_segments], (u32)(it % a.emit_segments), seg_units, lane);
      grid.sync();
      u32* s_segbase = s_hist;
      // a team of blocks per worker (all workers at once while there are at most as many as blocks)
      const int64_t teams = nf < (int64_t)gridDim.x ? (int64_t)gridDim.x / nf : 1;
      const int64_t slots = (int64_t)gridDim.x / teams;
      const u32 member = (u32)(blockIdx.x % teams);
      for (int64_t f = blockIdx.x / teams; f < nf; f += slots) {  // the same in every thread of the block
        const int n = (int)s_flagged[f];
        constexpr int kSegPer = kMaxSegments / kDenseThreads;  // consecutive mask segments per thread
        u32 mine[kSegPer], sum = 0, total;
#pragma unroll
        for (int i = 0; i < kSegPer; ++i) {
          const u32 sg = (u32)(kSegPer * tid + i);
          mine[i] = sg < a.emit_segments ? __ldcg(&p.segtot[(size_t)n * kMaxSegments + sg]) : 0u;
          sum += mine[i];
        }
        u32 base = block_excl_scan(sum, s_scan, &total);
        __syncthreads();
#pragma unroll
        for (int i = 0; i < kSegPer; ++i) {
          const u32 sg = (u32)(kSegPer * tid + i);
          if (sg < a.emit_segments) {
            s_segbase[sg] = base;
            if (member == 0u) p.segbase[(size_t)n * kMaxSegments + sg] = base;  // for k_aggregate
          }
          base += mine[i];
        }
        __syncthreads();
        if (total != k) {
          if (member == 0u && tid == 0) atomicOr(&p.gctl->err, kErrCountMismatch);
        } else {
          post_emit(p, n, member * blockDim.x + tid, (u32)teams * blockDim.x, 0u, 0u, true, 0u, 0u, 0u, s_segbase, seg_units);
        }
        __syncthreads();
      }
    }
    grid.sync();  // everyone has read the flag word before it is cleared for the next group and the next launch
    if (blockIdx.x == 0 && tid == 0) p.gctl->dense_flags = 0u;
  }
}

// ---------------------------------------------------------------------------------------------
// k_aggregate: g = sum_n omega_n * ghat_n with the workers added in the order n = 0..N-1.
// One thread per pair sent this round: the pair of the highest-numbered worker that sent index j
// owns g[j]; it looks the lower workers' values up (mask quad, prefix counts, value) and adds them
// in order.  One thread per pair of the previous round clears g[j] if nobody sent j now.
// ---------------------------------------------------------------------------------------------
struct AggArgs {
  float* g;
  int64_t d;
  int N;
  int64_t k;
  const int32_t* cur_idx;
  const float* cur_val;
  const int32_t* prev_idx;
  const u32* bitmask;
  const u32* qprefix;
  const u32* segbase;
  int64_t seg_units;
  int64_t W;
  const float* omega;
  int has_prev;
  float* theta;  // optional model vector: theta[j] <- theta[j] - eta * g[j] where g[j] was written
  float eta;
  float* num;    // [N][k] out: g[j] - omega_n * a_n[j] for every pair of this round: the numerator of next round's
                 // distortion (Eq. (Delta_def)), formed here where g[j] has just been summed; or NULL
};

__global__ void __launch_bounds__(256) k_aggregate(AggArgs p) {
  // grid: x over the pairs of one worker, y = worker, z = 0 for this round's pairs, 1 for the previous round's
  const int64_t Q = p.W >> 2;
  const int n = blockIdx.y;
  const bool prev_pass = blockIdx.z != 0;
  const u32 seg_units = (u32)p.seg_units;
  grid_dependency_begin();
  for (int64_t r = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; r < p.k; r += (int64_t)gridDim.x * blockDim.x) {
    const int64_t t = (int64_t)n * p.k + r;
    if (prev_pass) {  // a pair of the previous round
      const int32_t j = p.prev_idx[t];
      if (!RT_INB(j >= 0 && (int64_t)j < p.d)) continue;
      const size_t wi = (size_t)(j >> 5);
      const u32 bm = 1u << (j & 31);
      u32 any = 0;
      for (int m0 = 0; m0 < p.N; m0 += 8) {
        u32 w[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) w[u] = m0 + u < p.N ? p.bitmask[(size_t)(m0 + u) * p.W + wi] : 0u;
#pragma unroll
        for (int u = 0; u < 8; ++u) any |= w[u];
      }
      if (!(any & bm)) p.g[j] = 0.0f;
      continue;
    }
    const int32_t j = p.cur_idx[t];
    if (!RT_INB(j >= 0 && (int64_t)j < p.d)) continue;
    const size_t wi = (size_t)(j >> 5);
    const size_t qi = wi >> 2;
    const int wsub = (int)(wi & 3);
    const u32 bm = 1u << (j & 31);
    const size_t seg = (size_t)((u32)(wi >> 3) / seg_units);
    if (!RT_INB(seg < (size_t)kMaxSegments)) continue;
    // a higher-numbered worker that sent j owns it
    bool owned = true;
    for (int m0 = n + 1; m0 < p.N && owned; m0 += 8) {
      u32 w[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) w[u] = m0 + u < p.N ? p.bitmask[(size_t)(m0 + u) * p.W + wi] : 0u;
#pragma unroll
      for (int u = 0; u < 8; ++u) owned = owned && !(w[u] & bm);
    }
    if (!owned) continue;
    float sum = 0.0f;
    int contributors = 0;
    for (int m0 = 0; m0 < n; m0 += 4) {
      uint4 x[4];
      u32 pre[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const bool in = m0 + u < n;
        x[u] = in ? *reinterpret_cast<const uint4*>(p.bitmask + (size_t)(m0 + u) * p.W + qi * 4)
                  : make_uint4(0, 0, 0, 0);
        pre[u] = in ? p.qprefix[(size_t)(m0 + u) * Q + qi] + p.segbase[(size_t)(m0 + u) * kMaxSegments + seg] : 0u;
      }
      float v[4];
      bool has[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const u32 w[4] = {x[u].x, x[u].y, x[u].z, x[u].w};
        u32 rank = pre[u], mine = 0;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          if (i < wsub) rank += __popc(w[i]);
          if (i == wsub) mine = w[i];
        }
        has[u] = (mine & bm) != 0u;
        rank += __popc(mine & (bm - 1u));
        if (has[u] && !RT_INB((int64_t)rank < p.k)) has[u] = false;
        v[u] = has[u] ? p.cur_val[(size_t)(m0 + u) * p.k + rank] : 0.0f;
      }
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (has[u]) {
          sum = __fadd_rn(sum, __fmul_rn(p.omega[m0 + u], v[u]));
          ++contributors;
        }
    }
    const float own = p.cur_val[t];
    sum = __fadd_rn(sum, __fmul_rn(p.omega[n], own));
    p.g[j] = sum;
    if (p.num) p.num[t] = __fsub_rn(sum, __fmul_rn(p.omega[n], own));
    if (p.num && contributors) {  // the lower workers that sent j get theirs from here: their own pairs' threads do not own g[j]
      for (int m = 0; m < n; ++m) {
        const uint4 x = *reinterpret_cast<const uint4*>(p.bitmask + (size_t)m * p.W + qi * 4);
        const u32 w[4] = {x.x, x.y, x.z, x.w};
        u32 mine = 0, rank = 0;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          if (i < wsub) rank += __popc(w[i]);
          if (i == wsub) mine = w[i];
        }
        if (!(mine & bm)) continue;
        rank += p.qprefix[(size_t)m * Q + qi] + p.segbase[(size_t)m * kMaxSegments + seg] + __popc(mine & (bm - 1u));
        if (!RT_INB((int64_t)rank < p.k)) continue;
        const size_t tm = (size_t)m * p.k + rank;
        p.num[tm] = __fsub_rn(sum, __fmul_rn(p.omega[m], p.cur_val[tm]));
      }
    }
    // theta - eta * 0 is theta, so updating only where the aggregate is non-trivial is the dense update
    if (p.theta) p.theta[j] = __fsub_rn(p.theta[j], __fmul_rn(p.eta, sum));
  }
}

// ---------------------------------------------------------------------------------------------
// Aggregation over gathered pairs (regtopk_aggregate_gathered): the workers are spread over several GPUs, every GPU
// has all workers' pairs after an all-gather and adds them into its own cleared g, one launch per worker in worker
// order.  Within a worker the indices are distinct, so a launch has no two threads on one g[j], and the stream
// orders the launches: g[j] = (((0 + w_0 v_0) + w_1 v_1) + ...) exactly as the server sum is defined.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) k_scatter_add(float* g, int64_t d, int64_t k, const int32_t* idx, const float* val,
                                                     float omega) {
  for (int64_t r = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; r < k; r += (int64_t)gridDim.x * blockDim.x) {
    const int32_t j = idx[r];
    if ((u32)j >= (u32)d) continue;  // gathered data is not the library's own: an index out of range is ignored
    g[j] = __fadd_rn(g[j], __fmul_rn(omega, val[r]));
  }
}

// ---------------------------------------------------------------------------------------------
// Aggregation from explicit pairs with built-in scratch (regtopk_aggregate_pairs_static).
// The scratch is a file-scope device array: it costs 8 MiB on every GPU that loads this library,
// and it is shared by all calls on that GPU.  Host code never uses the symbol as a pointer; it asks
// the runtime for the array's device address once per device.
// ---------------------------------------------------------------------------------------------
static __device__ __align__(256) u32 g_static_scratch[REGTOPK_STATIC_SCRATCH_WORDS];

struct StaticAggArgs {
  float* g;
  int64_t d;
  int N;
  int64_t k;
  const int32_t* idx;
  const float* val;
  u32* mask;  // [N][W], inside the static scratch, cleared by the caller of the kernels
  int64_t W;
  float omega[REGTOPK_STATIC_MAX_WORKERS];
};

// The pairs come from the caller, not from the library's own selection, so every index is tested against
// [0, d) before it addresses the scratch or g; a pair that fails is ignored (the checked build counts it).
__device__ __forceinline__ bool static_index_ok(int32_t j, int64_t d) {
  if ((u32)j < (u32)d) return true;
#if REGTOPK_DEBUG
  atomicAdd(&g_bounds_faults, 1u);
#endif
  return false;
}

__global__ void __launch_bounds__(256) k_static_mark(StaticAggArgs p) {
  const int64_t total = p.k * p.N;
  for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < total;
       t += (int64_t)gridDim.x * blockDim.x) {
    const int n = (int)(t / p.k);
    const int32_t j = p.idx[t];
    if (!static_index_ok(j, p.d)) continue;
    atomicOr(&p.mask[(size_t)n * p.W + ((u32)j >> 5)], 1u << (j & 31));
  }
}

// Same ownership rule as k_aggregate (the highest-numbered worker that sent j writes g[j], adding the
// lower workers' terms in order); a lower worker's value is found by binary search in its ascending
// index row instead of through the prefix directory a context keeps.
__global__ void __launch_bounds__(256) k_static_aggregate(StaticAggArgs p) {
  const int64_t total = p.k * p.N;
  for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < total;
       t += (int64_t)gridDim.x * blockDim.x) {
    const int n = (int)(t / p.k);
    const int32_t j = p.idx[t];
    if (!static_index_ok(j, p.d)) continue;
    const size_t wi = (size_t)((u32)j >> 5);
    const u32 bm = 1u << (j & 31);
    bool owned = true;
    for (int m = n + 1; m < p.N && owned; ++m) owned = !(p.mask[(size_t)m * p.W + wi] & bm);
    if (!owned) continue;
    float sum = 0.0f;
    for (int m = 0; m < n; ++m) {
      if (!(p.mask[(size_t)m * p.W + wi] & bm)) continue;
      const int32_t* row = p.idx + (size_t)m * p.k;
      int64_t lo = 0, hi = p.k;
      while (lo < hi) {
        const int64_t mid = (lo + hi) >> 1;
        if (row[mid] < j) lo = mid + 1; else hi = mid;
      }
      // rows that are not ascending can send the search past the entry: such a term is left out
      if (lo < p.k && row[lo] == j) sum = __fadd_rn(sum, __fmul_rn(p.omega[m], p.val[(size_t)m * p.k + lo]));
    }
    sum = __fadd_rn(sum, __fmul_rn(p.omega[n], p.val[t]));
    p.g[j] = sum;
  }
}

// ---------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------
inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct Layout {
  int64_t ld, W, capA, stride;
  int64_t n_seg, tiles;  // segments of a row (layers; 1 in the plain mode) and k_dense tiles per row
  int64_t cuts;          // entries per row of the layer-wise cutoff table
  size_t off_chunk_cut;
  size_t off_dhist, off_seg_thr, off_seg, off_tile_ties, off_seg_end, off_seg_kpre, off_seg_tile0;
  size_t off_eps, off_g, off_mask[2], off_ctl, off_gctl, off_shist, zero_end, off_skeys, off_qprefix, off_segtot, off_segbase, off_ghist, off_btot, off_idx[2], off_val[2],
      off_ovr_key, off_ovr_comp, off_candA, off_candB, off_num[2], off_omega, off_stage_g, off_stage_idx,
      off_stage_val, total;
};

bool valid_problem(int64_t d, int32_t N, int64_t k, const regtopk_params* pr) {
  if (!pr) return false;
  if (d < 1 || d > 2147483646LL || N < 1 || N > 65535 || k < 1 || k > d) return false;
  if (!(pr->mu >= 0.0f) || !isfinite(pr->mu)) return false;
  if (!(pr->y >= 0.0f && pr->y <= 1.0f)) return false;  // 0 means "not set": y = 1
  if (pr->grad_dtype != REGTOPK_GRAD_F32 && pr->grad_dtype != REGTOPK_GRAD_BF16) return false;
  if (pr->omega)
    for (int n = 0; n < N; ++n)
      if (!isfinite(pr->omega[n])) return false;
  if (pr->n_layers < 0 || pr->n_layers > 65536) return false;
  if (pr->n_layers > 0) {  // contiguous layers that cover [0, d); the per-layer k add up to k
    if (!pr->layer_end || !pr->layer_k) return false;
    int64_t begin = 0, ksum = 0;
    for (int l = 0; l < pr->n_layers; ++l) {
      if (pr->layer_end[l] <= begin || pr->layer_end[l] > d) return false;
      if (pr->layer_k[l] < 1 || pr->layer_k[l] > pr->layer_end[l] - begin) return false;
      ksum += pr->layer_k[l];
      begin = pr->layer_end[l];
    }
    if (begin != d || ksum != k) return false;
  }
  return true;
}

// Segment tables of k_dense on the host: ends, exclusive prefix sums of the per-segment k, first tile of each
// segment (tiles of kDenseTile coordinates never straddle a segment).  Arrays of n_seg, n_seg + 1, n_seg + 1.
int64_t segment_tables(int64_t d, int64_t k, const regtopk_params* pr, int64_t* seg_end, int64_t* seg_kpre,
                       int64_t* seg_tile0) {
  const int64_t n_seg = pr->n_layers > 0 ? pr->n_layers : 1;
  int64_t begin = 0, kpre = 0, tile = 0;
  for (int64_t s = 0; s < n_seg; ++s) {
    const int64_t end = pr->n_layers > 0 ? pr->layer_end[s] : d;
    const int64_t ks = pr->n_layers > 0 ? pr->layer_k[s] : k;
    if (seg_end) { seg_end[s] = end; seg_kpre[s] = kpre; seg_tile0[s] = tile; }
    kpre += ks;
    tile += (end - begin + kDenseTile - 1) / kDenseTile;
    begin = end;
  }
  if (seg_end) { seg_kpre[n_seg] = kpre; seg_tile0[n_seg] = tile; }
  return tile;
}

Layout make_layout(int64_t d, int32_t N, int64_t k, const regtopk_params* pr) {
  Layout L;
  L.ld = (int64_t)align_up((size_t)d, 1024);
  L.W = (int64_t)align_up((size_t)((d + 31) / 32), 32);
  const int64_t M = d < kSampleMax ? d : kSampleMax;
  const int64_t kt = pr->mu > 0.0f ? (2 * k < d ? 2 * k : d) : k;
  int64_t cap = 3 * kt + 64 * ((d + M - 1) / M) + 4096;
  // layer-wise mode gathers by per-layer bounds that are a coarse bin edge below each layer's threshold: room for
  // many times k (measured 17-22 k on the ResNet-18 tensor table)
  if (pr->n_layers > 0 && cap < 48 * k + 4096) cap = 48 * k + 4096;
  if (cap > d) cap = d;
  if (cap < k) cap = k;
  L.capA = cap;
  L.stride = cap + k;
  size_t o = 0;
  auto take = [&](size_t bytes) { size_t at = o; o = align_up(o + bytes, 256); return at; };
  // state that creation and reset clear to zero comes first
  L.off_eps = take((size_t)N * L.ld * 4);
  L.off_g = take(align_up((size_t)d, 64) * 4);
  L.off_mask[0] = take((size_t)N * L.W * 4);
  L.off_mask[1] = take((size_t)N * L.W * 4);
  L.off_ctl = take((size_t)N * sizeof(WorkerCtl));
  L.off_gctl = take(sizeof(GlobalCtl));
  L.off_shist = take((size_t)N * kSampleBins * 4);
  L.n_seg = pr->n_layers > 0 ? pr->n_layers : 1;
  L.tiles = segment_tables(d, k, pr, nullptr, nullptr, nullptr);
  L.off_dhist = take((size_t)N * L.n_seg * kBins * 4);
  L.off_seg_thr = take((size_t)N * L.n_seg * 4);
  L.zero_end = o;
  L.off_seg = take((size_t)N * L.n_seg * sizeof(SegState));
  L.off_tile_ties = take((size_t)N * L.tiles * 8);
  L.off_seg_end = take((size_t)L.n_seg * 8);
  L.off_seg_kpre = take((size_t)(L.n_seg + 1) * 8);
  L.off_seg_tile0 = take((size_t)(L.n_seg + 1) * 8);
  L.cuts = (d + kCutSpan - 1) / kCutSpan;
  L.off_chunk_cut = take(pr->n_layers > 0 ? (size_t)N * L.cuts * 4 : 0);
  L.off_skeys = take((size_t)N * kSampleMax * 4);
  L.off_qprefix = take((size_t)N * (L.W / 4) * 4);
  L.off_segtot = take((size_t)N * kMaxSegments * 4);
  L.off_segbase = take((size_t)N * kMaxSegments * 4);
  L.off_ghist = take((size_t)N * 4 * kBins * 4);
  L.off_btot = take((size_t)N * 2 * kMaxCluster * 4);
  for (int i = 0; i < 2; ++i) {
    L.off_idx[i] = take((size_t)N * k * 4);
    L.off_val[i] = take((size_t)N * k * 4);
  }
  L.off_ovr_key = take((size_t)N * k * 4);
  L.off_ovr_comp = take((size_t)N * k * 8);
  L.off_candA = take((size_t)N * L.stride * 8);
  L.off_candB = take((size_t)N * L.stride * 8);
  for (int i = 0; i < 2; ++i) L.off_num[i] = take((size_t)N * k * 4);
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
#ifndef REGTOPK_MANY_PAIRS
#define REGTOPK_MANY_PAIRS 262144
#endif
constexpr int64_t kManyPairs = REGTOPK_MANY_PAIRS;  // N*k from which the list phases run in wide mode
constexpr int64_t kNumFromAggregate = 1ll << 26;    // d from which k_aggregate forms the next round's numerators
constexpr int64_t kGridDenseCoords = 1ll << 28;     // N*d from which the dense exact path runs on the whole grid

}  // namespace

struct regtopk_ctx {
  int64_t d, k;
  int32_t N;
  float mu, inv_y;
  int32_t grad_dtype, flags;
  Layout L;
  char* ws;
  cudaStream_t stream;
  int cur;           // which pair buffer receives this round's pairs
  int64_t round;
  int stepped;       // worker_step done, aggregate pending
  int sticky;        // first CUDA error seen
  int num_sms;
  int cluster;       // blocks per worker in k_post
  int many_pairs;    // N*k is large (or the testing flag is set): wide kernels and pair-mode emission
  int num_valid;     // the numerators of the previous pairs (off_num[prev]) were written by the last aggregation
  int layered;       // one selection per layer: every worker takes the dense path of k_dense every round
  int grid_dense;    // workers that need the dense exact path are served by k_dense, not by their k_post cluster
  int dense_blocks;  // co-resident blocks of k_dense (its grid)
  uint64_t layer_hash;
  int stream_blocks[5];
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

size_t sample_smem() { return (size_t)kSamplePadded * sizeof(u32); }
size_t dense_smem() { return (size_t)2 * kDenseWarps * kWarpList * sizeof(u64); }

// Launch configuration: `blocks` blocks of `threads`, optionally in clusters, always with programmatic
// stream serialization (see grid_dependency_begin).  attr must have room for two attributes.
void launch_config(cudaLaunchConfig_t* cfg, cudaLaunchAttribute* attr, unsigned blocks, int cluster,
                   int threads, size_t smem, cudaStream_t s) {
  memset(cfg, 0, sizeof *cfg);
  cfg->gridDim = dim3(blocks, 1, 1);
  cfg->blockDim = dim3((unsigned)threads, 1, 1);
  cfg->dynamicSmemBytes = smem;
  cfg->stream = s;
  int na = 0;
  attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[na].val.programmaticStreamSerializationAllowed = 1;
  ++na;
  if (cluster > 1) {
    attr[na].id = cudaLaunchAttributeClusterDimension;
    attr[na].val.clusterDim.x = (unsigned)cluster;
    attr[na].val.clusterDim.y = 1;
    attr[na].val.clusterDim.z = 1;
    ++na;
  }
  cfg->attrs = attr;
  cfg->numAttrs = na;
}

template <bool BF16, bool VEC, bool INPLACE = false>
void launch_stream(regtopk_ctx* c, const StreamArgs& a, int variant) {
  if (c->stream_blocks[variant] == 0) {
    int per_sm = 0;
    cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_stream<BF16, VEC, INPLACE>, kStreamThreads, 0);
    if (per_sm < 1) per_sm = 1;
    c->stream_blocks[variant] = per_sm * c->num_sms;
  }
  const int64_t chunk = StreamShape<BF16, VEC, INPLACE>::kChunk;
  const int64_t chunks = ((a.d + chunk - 1) / chunk) * a.N;
  int64_t blocks = (chunks + (kStreamThreads / 32) - 1) / (kStreamThreads / 32);
  if (blocks > c->stream_blocks[variant]) blocks = c->stream_blocks[variant];
  cudaLaunchConfig_t cfg;
  cudaLaunchAttribute attr[2];
  launch_config(&cfg, attr, (unsigned)blocks, 1, kStreamThreads, 0, c->stream);
  cudaLaunchKernelEx(&cfg, k_stream<BF16, VEC, INPLACE>, a);
}

void post_config(cudaLaunchConfig_t* cfg, cudaLaunchAttribute* attr, int N, int cluster, int threads,
                 cudaStream_t s) {
  launch_config(cfg, attr, (unsigned)(N * cluster), cluster, threads, 0, s);
}

// Blocks per worker for k_post: the largest cluster size up to 16 (sizes above 8 need the
// non-portable opt-in) for which the device keeps all N clusters resident at once; failing that,
// the largest size it can schedule at all.
int choose_cluster(int N) {
  cudaFuncSetAttribute(k_post, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
  cudaGetLastError();
  int schedulable = 1;
  for (int cs = kMaxCluster; cs > 1; --cs) {  // any size, not only powers of two: 10 blocks for N = 8 on a B200
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr[2];
    post_config(&cfg, attr, N, cs, kBlockPost, nullptr);
    int nclusters = 0;
    if (cudaOccupancyMaxActiveClusters(&nclusters, k_post, &cfg) != cudaSuccess) {
      cudaGetLastError();
      continue;
    }
    if (nclusters >= N) return cs;  // all workers' clusters run at once
    if (nclusters >= 1 && schedulable == 1) schedulable = cs;
  }
  return schedulable;
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
    case REGTOPK_ERR_TOO_LARGE: return "problem exceeds the built-in static capacity (use a context with a workspace)";
    default: return "unknown error code";
  }
}

size_t regtopk_workspace_bytes(int64_t d, int32_t N, int64_t k, const regtopk_params* params) {
  if (!valid_problem(d, N, k, params)) return 0;
  return make_layout(d, N, k, params).total;
}

int regtopk_state_reset(regtopk_ctx* c) {
  if (!c) return REGTOPK_ERR_INVALID_ARG;
  // The device's error word lives in the memory cleared below: an error it holds becomes the context's sticky
  // code first, so that a reset cannot lose it (this read synchronises the stream; resets are rare).
  if (c->round > 0 || c->stepped) {
    GlobalCtl h;
    memset(&h, 0, sizeof h);
    if (cudaMemcpyAsync(&h, c->ws + c->L.off_gctl, sizeof h, cudaMemcpyDeviceToHost, c->stream) == cudaSuccess &&
        cudaStreamSynchronize(c->stream) == cudaSuccess && h.err && !c->sticky)
      c->sticky = REGTOPK_ERR_INTERNAL;
  }
#if REGTOPK_DEBUG
  {
    const unsigned int zero = 0;
    cudaMemcpyToSymbolAsync(g_nonfinite, &zero, sizeof zero, 0, cudaMemcpyHostToDevice, c->stream);
  }
#endif
  int rc = note_cuda(c, cudaMemsetAsync(c->ws, 0, c->L.zero_end, c->stream));
  c->round = 0;
  c->stepped = 0;
  c->cur = 0;
  c->num_valid = 0;
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
  c->inv_y = (params->y == 0.0f || params->y == 1.0f) ? 1.0f : 1.0f / params->y;
  c->grad_dtype = params->grad_dtype;
  c->flags = params->flags;
  c->L = L;
  c->ws = static_cast<char*>(workspace);
  c->stream = static_cast<cudaStream_t>(cuda_stream);
  c->num_sms = sms > 0 ? sms : 148;
  c->cluster = choose_cluster(N);
  c->many_pairs = (k * (int64_t)N >= kManyPairs || (params->flags & REGTOPK_FLAG_FORCE_WIDE_LISTS)) ? 1 : 0;
  c->layered = params->n_layers > 0 ? 1 : 0;
  // Rows large enough for one more (empty) kernel per round to go unnoticed get the full-grid dense path; on small
  // problems a worker's own cluster scans its row, which costs the common round nothing.
  c->grid_dense = (c->layered || c->many_pairs || (params->flags & REGTOPK_FLAG_GRID_DENSE_SELECT) ||
                   d * (int64_t)N >= kGridDenseCoords) ? 1 : 0;
  {
    int per_sm = 0;
    const void* dense_fn = c->layered ? (const void*)k_dense<true> : (const void*)k_dense<false>;
    if (cudaFuncSetAttribute(dense_fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dense_smem()) != cudaSuccess ||
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, dense_fn, kDenseThreads, dense_smem()) != cudaSuccess ||
        per_sm < 1) {
      cudaGetLastError();
      per_sm = 1;
    }
    int64_t blocks = (int64_t)per_sm * c->num_sms;
    if (blocks > (int64_t)N * L.tiles) blocks = (int64_t)N * L.tiles;
    c->dense_blocks = (int)(blocks < 1 ? 1 : blocks);
  }
  float* om = static_cast<float*>(malloc(sizeof(float) * N));
  if (!om) { free(c); return REGTOPK_ERR_INVALID_ARG; }
  for (int n = 0; n < N; ++n) om[n] = params->omega ? params->omega[n] : 1.0f / (float)N;
  int rc = regtopk_state_reset(c);
  // pageable source: the copy is staged before the call returns, so om may be freed right away
  if (rc == REGTOPK_OK)
    rc = note_cuda(c, cudaMemcpyAsync(c->ws + L.off_omega, om, sizeof(float) * N,
                                      cudaMemcpyHostToDevice, c->stream));
  int64_t* seg = static_cast<int64_t*>(malloc(sizeof(int64_t) * (3 * (size_t)L.n_seg + 2)));
  if (!seg) { free(om); free(c); return REGTOPK_ERR_INVALID_ARG; }
  {
    int64_t* seg_end = seg;
    int64_t* seg_kpre = seg + L.n_seg;
    int64_t* seg_tile0 = seg + 2 * L.n_seg + 1;
    segment_tables(d, k, params, seg_end, seg_kpre, seg_tile0);
    uint64_t h = 1469598103934665603ull;  // FNV-1a over the layer table: a checkpoint must come from the same layers
    for (int64_t i = 0; i < L.n_seg; ++i)
      for (int64_t v : {seg_end[i], seg_kpre[i + 1]}) { h ^= (uint64_t)v; h *= 1099511628211ull; }
    c->layer_hash = params->n_layers > 0 ? h : 0;
    if (rc == REGTOPK_OK)
      rc = note_cuda(c, cudaMemcpyAsync(c->ws + L.off_seg_end, seg_end, 8 * (size_t)L.n_seg, cudaMemcpyHostToDevice, c->stream));
    if (rc == REGTOPK_OK)
      rc = note_cuda(c, cudaMemcpyAsync(c->ws + L.off_seg_kpre, seg_kpre, 8 * ((size_t)L.n_seg + 1), cudaMemcpyHostToDevice, c->stream));
    if (rc == REGTOPK_OK)
      rc = note_cuda(c, cudaMemcpyAsync(c->ws + L.off_seg_tile0, seg_tile0, 8 * ((size_t)L.n_seg + 1), cudaMemcpyHostToDevice, c->stream));
  }
  if (rc == REGTOPK_OK) rc = note_cuda(c, cudaStreamSynchronize(c->stream));
  free(om);
  free(seg);
  if (rc != REGTOPK_OK) { free(c); return rc; }
  *out = c;
  return REGTOPK_OK;
}

}  // extern "C"

namespace {
// One round of all workers.  grads == NULL: the accumulator rows already hold a (regtopk_worker_step_inplace).
int step_impl(regtopk_ctx* c, const void* grads, int64_t grad_ld, int32_t* out_idx, float* out_val) {
  if (c->stepped) return REGTOPK_ERR_SEQUENCE;
  const Layout& L = c->L;
  const bool inplace = grads == nullptr;
  if (inplace) {  // never dereferenced; keeps the row arithmetic of the sampling kernel on a real buffer
    grads = at<float>(c, L.off_eps);
    grad_ld = L.ld;
  }
  const bool bf16 = !inplace && c->grad_dtype == REGTOPK_GRAD_BF16;
  const bool has_prev = c->round >= 1;
  const bool use_marks = has_prev && c->mu > 0.0f;
  const int prev = c->cur ^ 1;
  const uintptr_t gaddr = reinterpret_cast<uintptr_t>(grads);
  const bool vec = bf16 ? (grad_ld % (REGTOPK_STREAM_EPL_BF16) == 0 && gaddr % (2 * REGTOPK_STREAM_EPL_BF16) == 0)
                        : (grad_ld % 4 == 0 && gaddr % 16 == 0);
  int rc = REGTOPK_OK;

  SampleArgs sa;
  sa.grads = grads; sa.grad_ld = grad_ld; sa.eps = at<float>(c, L.off_eps); sa.ld = L.ld; sa.d = c->d;
  sa.k = c->k;
  sa.k_target = use_marks ? (2 * c->k < c->d ? 2 * c->k : c->d) : c->k;
  sa.ctl = at<WorkerCtl>(c, L.off_ctl);
  sa.shist = at<u32>(c, L.off_shist);
  sa.skeys = at<u32>(c, L.off_skeys);
  sa.ghist = at<u32>(c, L.off_ghist);
  sa.N = c->N; sa.use_marks = use_marks; sa.g_prev = at<float>(c, L.off_g);
  sa.prev_idx = at<int32_t>(c, L.off_idx[prev]); sa.prev_val = at<float>(c, L.off_val[prev]);
  sa.prev_num = (use_marks && c->num_valid) ? at<float>(c, L.off_num[prev]) : nullptr;
  sa.omega = at<float>(c, L.off_omega); sa.mu = c->mu; sa.inv_y = c->inv_y; sa.ovr_key = at<u32>(c, L.off_ovr_key);
  sa.share_override = 0;
  sa.inplace = inplace ? 1 : 0;
  sa.force_dense = c->layered ? 1 : ((c->flags & REGTOPK_FLAG_FORCE_DENSE_SELECT) ? (c->grid_dense ? 2 : 1) : 0);
  {
    cudaLaunchConfig_t scfg;
    cudaLaunchAttribute sattr[2];
    int extra = use_marks ? (c->num_sms - c->N * kSampleCluster) / kSampleCluster : 0;  // override clusters
    if (use_marks && extra < 1) extra = 1;
    sa.share_override = use_marks && c->k * (int64_t)c->N > (int64_t)4 * extra * kSampleCluster * kBlockSel;
    post_config(&scfg, sattr, c->N + extra, kSampleCluster, kBlockSel, c->stream);
    scfg.dynamicSmemBytes = sample_smem();
    cudaError_t se = bf16 ? cudaLaunchKernelEx(&scfg, k_sample_cutoff<true>, sa)
                          : cudaLaunchKernelEx(&scfg, k_sample_cutoff<false>, sa);
    c->launches++;
    if (se != cudaSuccess) return note_cuda(c, se);
    if ((rc = note_cuda(c, cudaGetLastError()))) return rc;
  }

  StreamArgs st;
  st.grads = grads; st.grad_ld = grad_ld; st.eps = at<float>(c, L.off_eps); st.ld = L.ld; st.d = c->d;
  st.N = c->N; st.ctl = sa.ctl; st.cand = at<u64>(c, L.off_candA); st.cap = L.capA; st.stride = L.stride;
  st.marks = use_marks ? at<u32>(c, L.off_mask[prev]) : nullptr; st.W = L.W;
  st.chunk_cut = nullptr; st.cuts = L.cuts;
  if (c->layered) {
    st.chunk_cut = at<u32>(c, L.off_chunk_cut);
    int64_t blocks = (L.cuts * c->N + 255) / 256;
    if (blocks > (int64_t)c->num_sms * 8) blocks = (int64_t)c->num_sms * 8;
    cudaLaunchConfig_t lcfg;
    cudaLaunchAttribute lattr[2];
    launch_config(&lcfg, lattr, (unsigned)blocks, 1, 256, 0, c->stream);
    cudaLaunchKernelEx(&lcfg, k_layer_cutoffs, at<u32>(c, L.off_chunk_cut), L.cuts, c->d, (int)c->N, (int)L.n_seg,
                       (const int64_t*)at<int64_t>(c, L.off_seg_end), (const u32*)at<u32>(c, L.off_seg_thr));
    if ((rc = after_launch(c))) return rc;
  }
  const bool prof = c->profiling && c->n_events < kMaxProfile;
  if (prof) cudaEventRecord(c->ev0[c->n_events], c->stream);
  if (inplace) launch_stream<false, true, true>(c, st, 4);
  else if (bf16) { if (vec) launch_stream<true, true>(c, st, 3); else launch_stream<true, false>(c, st, 2); }
  else { if (vec) launch_stream<false, true>(c, st, 1); else launch_stream<false, false>(c, st, 0); }
  if (prof) cudaEventRecord(c->ev1[c->n_events++], c->stream);
  if ((rc = after_launch(c))) return rc;

  PostArgs pa;
  pa.ctl = sa.ctl; pa.gctl = at<GlobalCtl>(c, L.off_gctl); pa.eps = at<float>(c, L.off_eps); pa.ld = L.ld; pa.d = c->d; pa.k = c->k;
  pa.g_prev = at<float>(c, L.off_g);
  pa.prev_idx = at<int32_t>(c, L.off_idx[prev]); pa.prev_val = at<float>(c, L.off_val[prev]);
  pa.omega = at<float>(c, L.off_omega); pa.mu = c->mu;
  pa.ovr_key = at<u32>(c, L.off_ovr_key); pa.ovr_comp = at<u64>(c, L.off_ovr_comp);
  pa.candA = at<u64>(c, L.off_candA); pa.candB = at<u64>(c, L.off_candB); pa.capA = L.capA; pa.stride = L.stride;
  pa.ghist = at<u32>(c, L.off_ghist); pa.shist = at<u32>(c, L.off_shist); pa.btot = at<u32>(c, L.off_btot);
  pa.mask_old = at<u32>(c, L.off_mask[prev]); pa.mask_new = at<u32>(c, L.off_mask[c->cur]);
  pa.qprefix = at<u32>(c, L.off_qprefix); pa.segtot = at<u32>(c, L.off_segtot);
  pa.segbase = at<u32>(c, L.off_segbase); pa.W = L.W;
  pa.out_idx = out_idx; pa.out_val = out_val;
  pa.cur_idx = at<int32_t>(c, L.off_idx[c->cur]); pa.cur_val = at<float>(c, L.off_val[c->cur]);
  pa.use_marks = use_marks; pa.has_stale = c->round >= 2;
  pa.pair_mode = c->many_pairs;
  pa.wide = c->many_pairs;
  pa.grid_dense = c->grid_dense;
  // wide kernels: the grid's blocks split evenly over the workers (blockIdx.y = worker)
  cudaLaunchConfig_t wcfg;
  cudaLaunchAttribute wattr[2];
  {
    int bx = c->num_sms / c->N;
    if (bx < 1) bx = 1;
    launch_config(&wcfg, wattr, (unsigned)bx, 1, kBlockPost, 0, c->stream);
    wcfg.gridDim = dim3((unsigned)bx, (unsigned)c->N, 1);
  }
  if (pa.wide) {
    cudaLaunchKernelEx(&wcfg, k_wide_hist, pa);
    if ((rc = after_launch(c))) return rc;
    cudaLaunchKernelEx(&wcfg, k_wide_classify, pa);
    if ((rc = after_launch(c))) return rc;
  }
  cudaLaunchConfig_t cfg;
  cudaLaunchAttribute attr[2];
  post_config(&cfg, attr, c->N, c->cluster, kBlockPost, c->stream);
  cudaError_t le = cudaLaunchKernelEx(&cfg, k_post, pa);
  c->launches++;
  if (le != cudaSuccess) return note_cuda(c, le);
  if ((rc = note_cuda(c, cudaGetLastError()))) return rc;
  if (c->grid_dense) {
    // Cooperative launch in plain stream order: it starts when k_post has completed, and returns at once unless a
    // worker asked for the dense path.
    DenseArgs da;
    da.p = pa; da.N = c->N; da.n_seg = (int)L.n_seg; da.finish = pa.wide ? 0 : 1;
    da.emit_segments = c->layered ? (u32)kMaxSegments : (u32)(c->cluster * (kBlockPost / 32));
    da.tiles = L.tiles;
    da.seg_end = at<int64_t>(c, L.off_seg_end); da.seg_kpre = at<int64_t>(c, L.off_seg_kpre);
    da.seg_tile0 = at<int64_t>(c, L.off_seg_tile0);
    da.dhist = at<u32>(c, L.off_dhist); da.seg = at<SegState>(c, L.off_seg); da.tile_ties = at<u32>(c, L.off_tile_ties);
    da.seg_thr = at<u32>(c, L.off_seg_thr); da.layered = c->layered;
    cudaLaunchConfig_t dcfg;
    cudaLaunchAttribute dattr[1];
    memset(&dcfg, 0, sizeof dcfg);
    dcfg.gridDim = dim3((unsigned)c->dense_blocks, 1, 1);
    dcfg.blockDim = dim3(kDenseThreads, 1, 1);
    dcfg.dynamicSmemBytes = dense_smem();
    dcfg.stream = c->stream;
    dattr[0].id = cudaLaunchAttributeCooperative;
    dattr[0].val.cooperative = 1;
    dcfg.attrs = dattr;
    dcfg.numAttrs = 1;
    cudaError_t de = c->layered ? cudaLaunchKernelEx(&dcfg, k_dense<true>, da) : cudaLaunchKernelEx(&dcfg, k_dense<false>, da);
    c->launches++;
    if (de != cudaSuccess) return note_cuda(c, de);
    if ((rc = note_cuda(c, cudaGetLastError()))) return rc;
  }
  if (pa.wide) {
    cudaLaunchKernelEx(&wcfg, k_wide_prefix, pa);
    if ((rc = after_launch(c))) return rc;
    cudaLaunchKernelEx(&wcfg, k_wide_emit, pa);
    if ((rc = after_launch(c))) return rc;
  }
  if (pa.pair_mode) {
    UnzipArgs ua;
    ua.candB = pa.candB; ua.stride = L.stride; ua.k = c->k; ua.N = c->N;
    ua.out_idx = out_idx; ua.out_val = out_val; ua.cur_idx = pa.cur_idx; ua.cur_val = pa.cur_val;
    int64_t bx = (c->k + 255) / 256;
    const int64_t cap_x = ((int64_t)c->num_sms * 16 + c->N - 1) / c->N;
    if (bx > cap_x) bx = cap_x;
    cudaLaunchConfig_t ucfg;
    cudaLaunchAttribute uattr[2];
    launch_config(&ucfg, uattr, (unsigned)bx, 1, 256, 0, c->stream);
    ucfg.gridDim = dim3((unsigned)bx, (unsigned)c->N, 1);
    cudaLaunchKernelEx(&ucfg, k_unzip, ua);
    if ((rc = after_launch(c))) return rc;
  }

  c->stepped = 1;
  return REGTOPK_OK;
}
}  // namespace

extern "C" {

int regtopk_worker_step(regtopk_ctx* c, const void* grads, int64_t grad_ld, int32_t* out_idx,
                        float* out_val) {
  if (!c || !grads || !out_idx || !out_val || grad_ld < c->d) return REGTOPK_ERR_INVALID_ARG;
  return step_impl(c, grads, grad_ld, out_idx, out_val);
}

int regtopk_accumulator(regtopk_ctx* c, float** dev_ptr, int64_t* ld) {
  if (!c || !dev_ptr || !ld) return REGTOPK_ERR_INVALID_ARG;
  *dev_ptr = at<float>(c, c->L.off_eps);
  *ld = c->L.ld;
  return REGTOPK_OK;
}

int regtopk_worker_step_inplace(regtopk_ctx* c, int32_t* out_idx, float* out_val) {
  if (!c || !out_idx || !out_val) return REGTOPK_ERR_INVALID_ARG;
  return step_impl(c, nullptr, 0, out_idx, out_val);
}

int regtopk_aggregate(regtopk_ctx* c, float* out_g) { return regtopk_aggregate_update(c, nullptr, 0.0f, out_g); }

int regtopk_aggregate_update(regtopk_ctx* c, float* theta, float eta, float* out_g) {
  if (!c || (theta && !isfinite(eta))) return REGTOPK_ERR_INVALID_ARG;
  if (!c->stepped) return REGTOPK_ERR_SEQUENCE;
  const Layout& L = c->L;
  AggArgs a;
  a.g = at<float>(c, L.off_g); a.d = c->d; a.N = c->N; a.k = c->k;
  a.cur_idx = at<int32_t>(c, L.off_idx[c->cur]); a.cur_val = at<float>(c, L.off_val[c->cur]);
  a.prev_idx = at<int32_t>(c, L.off_idx[c->cur ^ 1]);
  a.bitmask = at<u32>(c, L.off_mask[c->cur]); a.qprefix = at<u32>(c, L.off_qprefix); a.segbase = at<u32>(c, L.off_segbase);
  {  // segments of the mask row as the emission cut them: one per warp of the k_post cluster; kMaxSegments in wide
     // mode and in layer-wise mode, where the whole grid emits
    const int64_t nseg = (c->many_pairs || c->layered) ? kMaxSegments : (int64_t)c->cluster * (kBlockPost / 32);
    a.seg_units = ((L.W >> 3) + nseg - 1) / nseg;
  }
  a.W = L.W;
  a.omega = at<float>(c, L.off_omega);
  a.has_prev = c->round >= 1;
  a.theta = theta; a.eta = eta;
  // Worth it where a gather from g misses the L2 cache (g of 256 MB and more): the next round's override pass then
  // reads the numerators in order instead (measured on the 1.3e9 shape at k = 1 %: 20.2 -> 19.0 ms per round).  On
  // small problems the extra stores and the second walk over the lower workers cost more than the gather saves
  // (ResNet-18 shape: 0.219 -> 0.230 ms).
  const bool form_num = c->d >= kNumFromAggregate || (c->flags & REGTOPK_FLAG_NUMERATORS_AT_AGGREGATE);
  a.num = form_num ? at<float>(c, L.off_num[c->cur]) : nullptr;
  {
    const int passes = a.has_prev ? 2 : 1;
    int64_t bx = (c->k + 255) / 256;
    const int64_t cap_x = ((int64_t)c->num_sms * 32 + (int64_t)c->N * passes - 1) / ((int64_t)c->N * passes);
    if (bx > cap_x) bx = cap_x;
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr[2];
    launch_config(&cfg, attr, (unsigned)bx, 1, 256, 0, c->stream);
    cfg.gridDim = dim3((unsigned)bx, (unsigned)c->N, (unsigned)passes);
    cudaLaunchKernelEx(&cfg, k_aggregate, a);
  }
  int rc = after_launch(c);
  if (rc) return rc;
  if (out_g)
    rc = note_cuda(c, cudaMemcpyAsync(out_g, a.g, (size_t)c->d * 4, cudaMemcpyDeviceToDevice, c->stream));
  c->cur ^= 1;  // this round's pairs are now "previous"
  c->round++;
  c->stepped = 0;
  c->num_valid = form_num ? 1 : 0;
  return rc;
}

int regtopk_aggregate_gathered(regtopk_ctx* c, int32_t n_total, const int32_t* all_idx, const float* all_val,
                               const float* omega_all, float* out_g) {
  if (!c || n_total < 1 || n_total > 65535 || !all_idx || !all_val) return REGTOPK_ERR_INVALID_ARG;
  if (omega_all)
    for (int n = 0; n < n_total; ++n)
      if (!isfinite(omega_all[n])) return REGTOPK_ERR_INVALID_ARG;
  if (!c->stepped) return REGTOPK_ERR_SEQUENCE;
  const Layout& L = c->L;
  float* g = at<float>(c, L.off_g);
  int rc = note_cuda(c, cudaMemsetAsync(g, 0, (size_t)c->d * 4, c->stream));
  if (rc) return rc;
  int64_t blocks = (c->k + 255) / 256;
  if (blocks > (int64_t)c->num_sms * 16) blocks = (int64_t)c->num_sms * 16;
  for (int n = 0; n < n_total; ++n) {
    const float w = omega_all ? omega_all[n] : 1.0f / (float)n_total;
    k_scatter_add<<<(unsigned)blocks, 256, 0, c->stream>>>(g, c->d, c->k, all_idx + (size_t)n * c->k,
                                                           all_val + (size_t)n * c->k, w);
    if ((rc = after_launch(c))) return rc;
  }
  if (out_g) rc = note_cuda(c, cudaMemcpyAsync(out_g, g, (size_t)c->d * 4, cudaMemcpyDeviceToDevice, c->stream));
  c->cur ^= 1;  // this round's own pairs are now "previous"
  c->round++;
  c->stepped = 0;
  c->num_valid = 0;  // the numerators were not formed: the next round gathers from g
  return rc;
}

int regtopk_global_gradient(regtopk_ctx* c, const float** dev_ptr) {
  if (!c || !dev_ptr) return REGTOPK_ERR_INVALID_ARG;
  *dev_ptr = at<float>(c, c->L.off_g);
  return REGTOPK_OK;
}

namespace {
struct StateHeader {
  uint64_t magic;
  int64_t d, k, ld, W, round;
  int32_t N, cur, grad_dtype;
  uint32_t mu_bits, inv_y_bits;
  uint64_t layer_hash;
};
constexpr uint64_t kStateMagic = 0x52544B5354415445ull;  // "RTKSTATE"
constexpr size_t kStateHeaderBytes = 256;
size_t state_part1(const Layout& L) { return L.off_ctl; }                      // residuals, g, both masks
size_t state_part2(const Layout& L) { return L.off_ovr_key - L.off_idx[0]; }   // both pair buffers
}  // namespace

size_t regtopk_state_bytes(regtopk_ctx* c) {
  if (!c) return 0;
  return kStateHeaderBytes + state_part1(c->L) + state_part2(c->L);
}

int regtopk_state_export(regtopk_ctx* c, void* dst, size_t bytes) {
  if (!c || !dst) return REGTOPK_ERR_INVALID_ARG;
  if (bytes < regtopk_state_bytes(c)) return REGTOPK_ERR_WORKSPACE_TOO_SMALL;
  if (c->stepped) return REGTOPK_ERR_SEQUENCE;
  char hdr[kStateHeaderBytes];
  memset(hdr, 0, sizeof hdr);
  StateHeader h;
  h.magic = kStateMagic; h.d = c->d; h.k = c->k; h.ld = c->L.ld; h.W = c->L.W; h.round = c->round;
  h.N = c->N; h.cur = c->cur; h.grad_dtype = c->grad_dtype;
  memcpy(&h.mu_bits, &c->mu, 4);
  memcpy(&h.inv_y_bits, &c->inv_y, 4);
  h.layer_hash = c->layer_hash;
  memcpy(hdr, &h, sizeof h);
  char* out = static_cast<char*>(dst);
  // the header is pageable host memory: the runtime stages it before cudaMemcpyAsync returns
  int rc = note_cuda(c, cudaMemcpyAsync(out, hdr, kStateHeaderBytes, cudaMemcpyHostToDevice, c->stream));
  if (!rc) rc = note_cuda(c, cudaMemcpyAsync(out + kStateHeaderBytes, c->ws, state_part1(c->L),
                                            cudaMemcpyDeviceToDevice, c->stream));
  if (!rc) rc = note_cuda(c, cudaMemcpyAsync(out + kStateHeaderBytes + state_part1(c->L), c->ws + c->L.off_idx[0],
                                            state_part2(c->L), cudaMemcpyDeviceToDevice, c->stream));
  return rc;
}

int regtopk_state_import(regtopk_ctx* c, const void* src, size_t bytes) {
  if (!c || !src) return REGTOPK_ERR_INVALID_ARG;
  if (bytes < regtopk_state_bytes(c)) return REGTOPK_ERR_WORKSPACE_TOO_SMALL;
  const char* in = static_cast<const char*>(src);
  StateHeader h;
  int rc = note_cuda(c, cudaMemcpyAsync(&h, in, sizeof h, cudaMemcpyDeviceToHost, c->stream));
  if (!rc) rc = note_cuda(c, cudaStreamSynchronize(c->stream));
  if (rc) return rc;
  uint32_t mu_bits, inv_y_bits;
  memcpy(&mu_bits, &c->mu, 4);
  memcpy(&inv_y_bits, &c->inv_y, 4);
  if (h.magic != kStateMagic || h.d != c->d || h.k != c->k || h.N != c->N || h.ld != c->L.ld || h.W != c->L.W ||
      h.grad_dtype != c->grad_dtype || h.mu_bits != mu_bits || h.inv_y_bits != inv_y_bits || h.layer_hash != c->layer_hash || h.round < 0 || (h.cur != 0 && h.cur != 1))
    return REGTOPK_ERR_INVALID_ARG;
  rc = regtopk_state_reset(c);  // clears the control blocks and histograms as well
  if (!rc) rc = note_cuda(c, cudaMemcpyAsync(c->ws, in + kStateHeaderBytes, state_part1(c->L),
                                            cudaMemcpyDeviceToDevice, c->stream));
  if (!rc) rc = note_cuda(c, cudaMemcpyAsync(c->ws + c->L.off_idx[0], in + kStateHeaderBytes + state_part1(c->L),
                                            state_part2(c->L), cudaMemcpyDeviceToDevice, c->stream));
  if (!rc) { c->round = h.round; c->cur = h.cur; c->stepped = 0; }
  return rc;
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
#if REGTOPK_DEBUG
  unsigned int faults = 0;
  if (cudaMemcpyFromSymbol(&faults, g_bounds_faults, sizeof faults) != cudaSuccess) return note_cuda(c, cudaErrorUnknown);
  if (faults) return REGTOPK_ERR_INTERNAL;
  unsigned int nonfinite = 0;
  if (cudaMemcpyFromSymbol(&nonfinite, g_nonfinite, sizeof nonfinite) != cudaSuccess) return note_cuda(c, cudaErrorUnknown);
  if (!h.err && nonfinite) return REGTOPK_ERR_INVALID_ARG;
#endif
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
    out->device_error_bits = (int64_t)h.err;
    out->post_cluster_blocks = c->cluster;
#if REGTOPK_DEBUG
    unsigned int faults = 0;
    if (cudaMemcpyFromSymbol(&faults, g_bounds_faults, sizeof faults) == cudaSuccess && faults)
      out->device_error_bits |= (int64_t)kErrBounds;
#endif
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

int regtopk_aggregate_pairs_static(int64_t d, int32_t N, int64_t k, const int32_t* idx, const float* val,
                                   const float* omega, float* out_g, void* cuda_stream) {
  if (d < 1 || d > 2147483646LL || N < 1 || k < 1 || k > d || !idx || !val || !out_g)
    return REGTOPK_ERR_INVALID_ARG;
  if (N > REGTOPK_STATIC_MAX_WORKERS) return REGTOPK_ERR_TOO_LARGE;
  const int64_t W = ((d + 31) / 32 + 3) / 4 * 4;
  if ((int64_t)N * W > (int64_t)REGTOPK_STATIC_SCRATCH_WORDS) return REGTOPK_ERR_TOO_LARGE;
  // Device address of the scratch array, looked up once per device with that device current.  The cache is
  // written with release and read with acquire order: threads that race here all store the same address.
  static std::atomic<u32*> scratch_of_device[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return REGTOPK_ERR_NO_DEVICE;
  u32* scratch = scratch_of_device[dev].load(std::memory_order_acquire);
  if (!scratch) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) {
      cudaGetLastError();
      return REGTOPK_ERR_NO_DEVICE;
    }
    scratch = static_cast<u32*>(ptr);
    scratch_of_device[dev].store(scratch, std::memory_order_release);
  }
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  StaticAggArgs a;
  a.g = out_g; a.d = d; a.N = N; a.k = k; a.idx = idx; a.val = val; a.mask = scratch; a.W = W;
  for (int n = 0; n < REGTOPK_STATIC_MAX_WORKERS; ++n) {
    a.omega[n] = n < N ? (omega ? omega[n] : 1.0f / (float)N) : 0.0f;
    if (n < N && !isfinite(a.omega[n])) return REGTOPK_ERR_INVALID_ARG;
  }
  // the array keeps the previous call's bits: clear the rows this call uses, and the whole output
  if (cudaMemsetAsync(a.mask, 0, (size_t)N * W * sizeof(u32), stream) != cudaSuccess ||
      cudaMemsetAsync(out_g, 0, (size_t)d * sizeof(float), stream) != cudaSuccess)
    return REGTOPK_ERR_CUDA;
  const int64_t total = k * (int64_t)N;
  int64_t blocks = (total + 255) / 256;
  if (blocks > 148 * 32) blocks = 148 * 32;
  k_static_mark<<<(unsigned)blocks, 256, 0, stream>>>(a);
  if (cudaGetLastError() != cudaSuccess) return REGTOPK_ERR_CUDA;
  k_static_aggregate<<<(unsigned)blocks, 256, 0, stream>>>(a);
  if (cudaGetLastError() != cudaSuccess) return REGTOPK_ERR_CUDA;
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
