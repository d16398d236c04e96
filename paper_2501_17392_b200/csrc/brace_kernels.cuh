// Device kernels of the BRACE ring-aggregation library (sm_100a).
//
// Every kernel here is bound by HBM bandwidth (about three integer operations
// per 4-byte element), so the design rules are: 128-bit coalesced accesses,
// many independent loads in flight per thread, streaming cache hints for data
// that is read once, and no re-reads of anything that can stay in registers.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace brace {

// ---------------------------------------------------------------------------
// Partition of the d coordinates into n sub-vectors (Section 2.2).
// ---------------------------------------------------------------------------
struct Part {
  int64_t d;   // coordinates
  int64_t G;   // granule
  int64_t Q;   // ceil(d / G)
  int n;       // clients == sub-vectors
  __host__ __device__ __forceinline__ int64_t begin(int j) const {
    int64_t b = G * (((int64_t)j * Q) / n);
    return b < d ? b : d;
  }
};

__device__ __forceinline__ int next_client(int c, int n) { return c + 1 == n ? 0 : c + 1; }

// Debug build (-DBRACE_DEBUG): every ring kernel checks, before it touches memory, that the sub-vector
// it was handed lies inside the buffers it will index (update rows, mailboxes, output rows) and that
// its client indices are in range.  A check that fails records its code in a status word the host
// reads with brace_debug_status, and the CTA skips the sub-vector (the checks are uniform over a CTA, so
// no barrier is left waiting): nothing traps, the context stays usable.  In the release build every
// check is the constant true.
enum { kDbgUpdateRow = 1, kDbgMailbox = 2, kDbgOutputRow = 3, kDbgClient = 4 };
#ifdef BRACE_DEBUG
__device__ int g_debug_status = 0;                   // code of the first violation since the last read
__device__ __forceinline__ bool debug_ok(bool cond, int code) {
  if (!cond) atomicCAS(&g_debug_status, 0, code);
  return cond;
}
#else
__device__ __forceinline__ bool debug_ok(bool, int) { return true; }
#endif

// Section 3 Phase I: element-wise sign.  NaN compares false both ways -> 0.
template <bool ZS>
__device__ __forceinline__ int sgn1(float x, int zs) {
  int s = (int)(x > 0.0f) - (int)(x < 0.0f);
  if (ZS) s = (x == 0.0f) ? zs : s;
  return s;
}

// Programmatic dependent launch: the per-hop kernels are launched so that the
// next hop's CTAs may start while the current hop drains.  pdl_wait() returns
// once every kernel launched before this one on the stream has completed and
// its writes are visible; before it a kernel may only read memory that no
// earlier kernel of the round writes (the update matrix, from hop 1 on: hop 0
// waits for the matrix's producer before it lets hop 1 start).
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// streaming (read-once) 128-bit load
__device__ __forceinline__ float4 ld_stream(const float* p) { return __ldcs(reinterpret_cast<const float4*>(p)); }

__device__ __forceinline__ void store4(int8_t* p, int a, int b, int c, int d) {
  *reinterpret_cast<char4*>(p) = make_char4((signed char)a, (signed char)b, (signed char)c, (signed char)d);
}
__device__ __forceinline__ void store4(int16_t* p, int a, int b, int c, int d) {
  *reinterpret_cast<short4*>(p) = make_short4((short)a, (short)b, (short)c, (short)d);
}
// same, with the streaming hint (written once, not read again by this kernel)
__device__ __forceinline__ void store4_stream(int8_t* p, int a, int b, int c, int d) {
  __stcs(reinterpret_cast<char4*>(p), make_char4((signed char)a, (signed char)b, (signed char)c, (signed char)d));
}
__device__ __forceinline__ void store4_stream(int16_t* p, int a, int b, int c, int d) {
  __stcs(reinterpret_cast<short4*>(p), make_short4((short)a, (short)b, (short)c, (short)d));
}
__device__ __forceinline__ void load4(const int8_t* p, int& a, int& b, int& c, int& d) {
  char4 v = *reinterpret_cast<const char4*>(p);
  a = v.x; b = v.y; c = v.z; d = v.w;
}
__device__ __forceinline__ void load4(const int16_t* p, int& a, int& b, int& c, int& d) {
  short4 v = *reinterpret_cast<const short4*>(p);
  a = v.x; b = v.y; c = v.z; d = v.w;
}

// ---------------------------------------------------------------------------
// Share-Reduce hop, sign rule (Section 3 Phase II; Phase I fused into the read).
// grid = (tiles over the longest sub-vector, n senders).  Vector variant: a CTA
// covers 256*VPT float4; every thread issues its VPT update loads (and mailbox
// loads) before it consumes any of them.
// ---------------------------------------------------------------------------
template <typename P, int VPT, bool ZS>
__global__ void __launch_bounds__(256)
rs_step_sign_kernel(Part pt, const float* __restrict__ U, int64_t ld, const P* __restrict__ mail_in,
                    P* __restrict__ mail_out, int64_t seg_pad, int step, int zs) {
  const int n = pt.n;
  const int c = blockIdx.y;
  const int r = next_client(c, n);
  int j = c - step;
  if (j < 0) j += n;
  const int64_t b = pt.begin(j), e = (j + 1 == n) ? pt.d : pt.begin(j + 1);
  const int64_t L = e - b;
  if (!(debug_ok(b >= 0 && b <= e && e <= pt.d && pt.d <= ld, kDbgUpdateRow) && debug_ok(L <= seg_pad, kDbgMailbox) &&
        debug_ok(r >= 0 && r < n && j >= 0 && j < n, kDbgClient)))
    return;
  const float* uc = U + (int64_t)c * ld + b;
  const float* ur = U + (int64_t)r * ld + b;
  const P* in = mail_in + (int64_t)c * seg_pad;
  P* out = mail_out + (int64_t)r * seg_pad;
  // Hop 0 lets the next hop start only after it has itself seen the producer of the update
  // matrix complete: hop 1 reads its updates before its own wait, and that wait covers hop 0 only.
  if (step == 0) pdl_wait();
  pdl_launch_dependents();
  if (VPT > 0) {
    constexpr int V = VPT > 0 ? VPT : 1;
    const int64_t base = (int64_t)blockIdx.x * (256 * V) + threadIdx.x;
    if (base * 4 >= L) return;
    float4 x[V], y[V];
    int a[V][4];
    bool full[V];
#pragma unroll
    for (int v = 0; v < V; ++v) {                  // own updates: independent of the previous hop
      const int64_t i = (base + v * 256) * 4;
      full[v] = i + 4 <= L;
      if (full[v]) {
        x[v] = ld_stream(ur + i);
        if (step == 0) y[v] = ld_stream(uc + i);
      }
    }
    if (step != 0) {
      pdl_wait();                                  // previous hop done: mailboxes readable, other set writable
#pragma unroll
      for (int v = 0; v < V; ++v) {
        const int64_t i = (base + v * 256) * 4;
        if (full[v]) load4(in + i, a[v][0], a[v][1], a[v][2], a[v][3]);
      }
    }
#pragma unroll
    for (int v = 0; v < V; ++v) {
      const int64_t i = (base + v * 256) * 4;
      if (full[v]) {
        if (step == 0) {
          a[v][0] = sgn1<ZS>(y[v].x, zs); a[v][1] = sgn1<ZS>(y[v].y, zs);
          a[v][2] = sgn1<ZS>(y[v].z, zs); a[v][3] = sgn1<ZS>(y[v].w, zs);
        }
        store4(out + i, a[v][0] + sgn1<ZS>(x[v].x, zs), a[v][1] + sgn1<ZS>(x[v].y, zs),
               a[v][2] + sgn1<ZS>(x[v].z, zs), a[v][3] + sgn1<ZS>(x[v].w, zs));
      } else {
        for (int64_t k = i; k < L; ++k) {         // ragged end of the last sub-vector
          const int s0 = (step == 0) ? sgn1<ZS>(uc[k], zs) : (int)in[k];
          out[k] = (P)(s0 + sgn1<ZS>(ur[k], zs));
        }
      }
    }
  } else {
    if (step != 0) pdl_wait();
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t < L) {
      int s0 = (step == 0) ? sgn1<ZS>(uc[t], zs) : (int)in[t];
      out[t] = (P)(s0 + sgn1<ZS>(ur[t], zs));
    }
  }
}

// Share-Reduce hop, plain sum (Section 2.2 Phase I): float32 adds in ring order.
template <bool VEC>
__global__ void __launch_bounds__(256)
rs_step_sum_kernel(Part pt, const float* __restrict__ U, int64_t ld, const float* __restrict__ mail_in,
                   float* __restrict__ mail_out, int64_t seg_pad, int step) {
  const int n = pt.n;
  const int c = blockIdx.y;
  const int r = next_client(c, n);
  int j = c - step;
  if (j < 0) j += n;
  const int64_t b = pt.begin(j), e = (j + 1 == n) ? pt.d : pt.begin(j + 1);
  const int64_t L = e - b;
  if (!(debug_ok(b >= 0 && b <= e && e <= pt.d && pt.d <= ld, kDbgUpdateRow) && debug_ok(L <= seg_pad, kDbgMailbox) &&
        debug_ok(r >= 0 && r < n && j >= 0 && j < n, kDbgClient)))
    return;
  const float* uc = U + (int64_t)c * ld + b;
  const float* ur = U + (int64_t)r * ld + b;
  const float* in = (step == 0) ? uc : mail_in + (int64_t)c * seg_pad;
  float* out = mail_out + (int64_t)r * seg_pad;
  const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (step == 0) pdl_wait();                        // see rs_step_sign_kernel
  pdl_launch_dependents();
  if (VEC) {
    const int64_t i = t * 4;
    if (i + 4 <= L) {
      float4 x = ld_stream(ur + i);
      if (step != 0) pdl_wait();
      float4 y = (step == 0) ? ld_stream(in + i) : *reinterpret_cast<const float4*>(in + i);
      float4 o;
      o.x = __fadd_rn(y.x, x.x); o.y = __fadd_rn(y.y, x.y); o.z = __fadd_rn(y.z, x.z); o.w = __fadd_rn(y.w, x.w);
      *reinterpret_cast<float4*>(out + i) = o;
    } else {
      if (step != 0) pdl_wait();
      for (int64_t k = i; k < L; ++k) out[k] = __fadd_rn(in[k], ur[k]);
    }
  } else {
    if (step != 0) pdl_wait();
    if (t < L) out[t] = __fadd_rn(in[t], ur[t]);
  }
}

// ---------------------------------------------------------------------------
// Consensus, Eq. (1): one thread per 32-bit output word of the owner's sub-vector.
// The map is bit = (S > lam) | (S < lam_lo): Eq. (1) uses lam_lo = INT_MIN (never
// true); the symmetric |S| > theta variant uses lam = theta, lam_lo = -theta.
// Words that straddle a sub-vector boundary (granule % 32 != 0) are
// read-modify-written; in one launch each row is written by one sub-vector only.
// ---------------------------------------------------------------------------
template <typename P>
__global__ void __launch_bounds__(256)
consensus_sign_kernel(Part pt, const P* __restrict__ mail, int64_t seg_pad, uint32_t* __restrict__ out,
                      int64_t out_ld, int lam, int lam_lo) {
  pdl_launch_dependents();
  pdl_wait();
  const int n = pt.n;
  const int c = blockIdx.y;
  const int j = next_client(c, n);
  const int64_t b = pt.begin(j), e = (j + 1 == n) ? pt.d : pt.begin(j + 1);
  if (b >= e) return;
  const int64_t w0 = b >> 5, w1 = (e + 31) >> 5;
  if (!(debug_ok(e - b <= seg_pad && e <= pt.d, kDbgMailbox) && debug_ok(w1 <= out_ld, kDbgOutputRow))) return;
  const int64_t w = w0 + (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (w >= w1) return;
  const int64_t k0 = (w << 5) > b ? (w << 5) : b;
  const int64_t k1 = ((w + 1) << 5) < e ? ((w + 1) << 5) : e;
  const P* src = mail + (int64_t)c * seg_pad;      // src[k - b] is coordinate k
  uint32_t bits = 0;
  if (k1 - k0 == 32 && ((k0 - b) & 15) == 0) {
    constexpr int NV = (int)(32 * sizeof(P) / 16);
    uint4 raw[NV];
#pragma unroll
    for (int q = 0; q < NV; ++q) raw[q] = reinterpret_cast<const uint4*>(src + (k0 - b))[q];
    const P* v = reinterpret_cast<const P*>(raw);
#pragma unroll
    for (int q = 0; q < 32; ++q) bits |= (uint32_t)(((int)v[q] > lam) | ((int)v[q] < lam_lo)) << q;
  } else {
    for (int64_t k = k0; k < k1; ++k) bits |= (uint32_t)(((int)src[k - b] > lam) | ((int)src[k - b] < lam_lo)) << (int)(k & 31);
  }
  const int lo = (int)(k0 & 31);
  int hi = (int)(k1 - (w << 5));                    // one past the last bit this sub-vector owns
  if (k1 == pt.d) hi = 32;                          // bits past d are padding: written as 0
  const uint32_t mask = (hi == 32 ? 0xffffffffu : ((1u << hi) - 1u)) & ~((1u << lo) - 1u);
  uint32_t* dst = out + (int64_t)c * out_ld + w;
  *dst = (mask == 0xffffffffu) ? bits : ((*dst & ~mask) | bits);
}

// Phase III under the plain-sum rule: identity, or division by n.
template <bool VEC>
__global__ void __launch_bounds__(256)
consensus_sum_kernel(Part pt, const float* __restrict__ mail, int64_t seg_pad, float* __restrict__ out,
                     int64_t out_ld, int mean) {
  pdl_launch_dependents();
  pdl_wait();
  const int n = pt.n;
  const int c = blockIdx.y;
  const int j = next_client(c, n);
  const int64_t b = pt.begin(j), e = (j + 1 == n) ? pt.d : pt.begin(j + 1);
  const int64_t L = e - b;
  if (!(debug_ok(L <= seg_pad && b <= e, kDbgMailbox) && debug_ok(e <= pt.d && pt.d <= out_ld, kDbgOutputRow))) return;
  const float* src = mail + (int64_t)c * seg_pad;
  float* dst = out + (int64_t)c * out_ld + b;
  const float fn = (float)n;
  const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (VEC) {
    const int64_t i = t * 4;
    if (i + 4 <= L) {
      float4 v = *reinterpret_cast<const float4*>(src + i);
      if (mean) { v.x = __fdiv_rn(v.x, fn); v.y = __fdiv_rn(v.y, fn); v.z = __fdiv_rn(v.z, fn); v.w = __fdiv_rn(v.w, fn); }
      *reinterpret_cast<float4*>(dst + i) = v;
    } else {
      for (int64_t k = i; k < L; ++k) dst[k] = mean ? __fdiv_rn(src[k], fn) : src[k];
    }
  } else {
    if (t < L) dst[t] = mean ? __fdiv_rn(src[t], fn) : src[t];
  }
}

// ---------------------------------------------------------------------------
// Share-Only hop (Section 3 Phase IV): row c -> row (c+1) mod n, one sub-vector.
// ---------------------------------------------------------------------------
// WPT = words per thread: 4 copies 128 bits at a time (needs 16-byte aligned rows
// and granule % 128 == 0); boundary words of a sub-vector are always masked.
template <int WPT>
__global__ void __launch_bounds__(256)
ag_step_bits_kernel(Part pt, uint32_t* out, int64_t out_ld, int step) {
  pdl_launch_dependents();
  pdl_wait();
  const int n = pt.n;
  const int c = blockIdx.y;
  const int r = next_client(c, n);
  int j = c + 1 - step;
  if (j < 0) j += n;
  if (j >= n) j -= n;
  const int64_t b = pt.begin(j), e = (j + 1 == n) ? pt.d : pt.begin(j + 1);
  if (b >= e) return;
  const int64_t w0 = b >> 5, w1 = (e + 31) >> 5;
  if (!(debug_ok(w1 <= out_ld && e <= pt.d, kDbgOutputRow) && debug_ok(r >= 0 && r < n && j >= 0 && j < n, kDbgClient)))
    return;
  const int64_t wt = w0 + ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * WPT;
  if (wt >= w1) return;
  const uint32_t* src = out + (int64_t)c * out_ld;
  uint32_t* dst = out + (int64_t)r * out_ld;
  if (WPT == 4 && (wt << 5) >= b && ((wt + 4) << 5) <= e) {      // four whole words inside the sub-vector
    *reinterpret_cast<uint4*>(dst + wt) = *reinterpret_cast<const uint4*>(src + wt);
    return;
  }
#pragma unroll
  for (int q = 0; q < WPT; ++q) {
    const int64_t w = wt + q;
    if (w >= w1) break;
    const int64_t k0 = (w << 5) > b ? (w << 5) : b;
    const int64_t k1 = ((w + 1) << 5) < e ? ((w + 1) << 5) : e;
    const int lo = (int)(k0 & 31);
    int hi = (int)(k1 - (w << 5));
    if (k1 == pt.d) hi = 32;
    const uint32_t mask = (hi == 32 ? 0xffffffffu : ((1u << hi) - 1u)) & ~((1u << lo) - 1u);
    const uint32_t v = src[w];
    dst[w] = (mask == 0xffffffffu) ? v : ((dst[w] & ~mask) | (v & mask));
  }
}

// All of Share-Only at once, for the fused round: every sub-vector is copied from
// its owner's row to the n-1 other rows.  One CTA moves 4 KB of a sub-vector's
// words (256 threads x 128 bits) to each row in turn, so every row receives long
// contiguous bursts instead of the 128-byte pieces a tile of the fused kernel
// could offer.  grid = (chunks over the longest sub-vector, n sub-vectors, groups of rows);
// needs granule % 128 == 0 and 16-byte aligned rows.
__global__ void __launch_bounds__(256)
ag_all_bits_kernel(Part pt, uint32_t* out, int64_t out_ld, int rows_per_group) {
  pdl_launch_dependents();
  pdl_wait();
  const int n = pt.n;
  const int j = blockIdx.y;
  const int owner = j == 0 ? n - 1 : j - 1;
  const int64_t b = pt.begin(j), e = (j + 1 == n) ? pt.d : pt.begin(j + 1);
  if (b >= e) return;
  const int64_t w0 = b >> 5, w1 = (e + 31) >> 5;
  if (!(debug_ok(w1 <= out_ld && e <= pt.d, kDbgOutputRow) && debug_ok(owner >= 0 && owner < n, kDbgClient))) return;
  const int64_t wt = w0 + ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * 4;
  if (wt >= w1) return;
  const int r0 = blockIdx.z * rows_per_group;
  const int r1 = r0 + rows_per_group < n ? r0 + rows_per_group : n;
  const uint32_t* src = out + (int64_t)owner * out_ld + wt;
  if (wt + 4 <= w1) {
    const uint4 v = *reinterpret_cast<const uint4*>(src);
    for (int row = r0; row < r1; ++row)
      if (row != owner) __stcs(reinterpret_cast<uint4*>(out + (int64_t)row * out_ld + wt), v);
  } else {
    for (int64_t w = wt; w < w1; ++w) {
      const uint32_t v = out[(int64_t)owner * out_ld + w];
      for (int row = r0; row < r1; ++row)
        if (row != owner) out[(int64_t)row * out_ld + w] = v;
    }
  }
}

// Share-Only at once for the plain-sum rule: every sub-vector is copied from its owner's row to the
// n-1 other rows, 4 KB (256 threads x 128 bits) of a sub-vector per CTA and row group.
// grid = (chunks over the longest sub-vector, n sub-vectors, groups of rows); needs granule % 4 == 0
// and 16-byte aligned rows.
__global__ void __launch_bounds__(256)
ag_all_f32_kernel(Part pt, float* out, int64_t out_ld, int rows_per_group) {
  pdl_launch_dependents();
  pdl_wait();
  const int n = pt.n;
  const int j = blockIdx.y;
  const int owner = j == 0 ? n - 1 : j - 1;
  const int64_t b = pt.begin(j), e = (j + 1 == n) ? pt.d : pt.begin(j + 1);
  if (!(debug_ok(b <= e && e <= pt.d && pt.d <= out_ld, kDbgOutputRow) && debug_ok(owner >= 0 && owner < n, kDbgClient)))
    return;
  const int64_t i = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * 4;
  if (b + i >= e) return;
  const int r0 = blockIdx.z * rows_per_group;
  const int r1 = r0 + rows_per_group < n ? r0 + rows_per_group : n;
  const float* src = out + (int64_t)owner * out_ld + b + i;
  if (b + i + 4 <= e) {
    const float4 v = ld_stream(src);
    for (int row = r0; row < r1; ++row)
      if (row != owner) __stcs(reinterpret_cast<float4*>(out + (int64_t)row * out_ld + b + i), v);
  } else {
    for (int64_t k = b + i; k < e; ++k) {
      const float v = out[(int64_t)owner * out_ld + k];
      for (int row = r0; row < r1; ++row)
        if (row != owner) out[(int64_t)row * out_ld + k] = v;
    }
  }
}

template <bool VEC>
__global__ void __launch_bounds__(256)
ag_step_f32_kernel(Part pt, float* out, int64_t out_ld, int step) {
  pdl_launch_dependents();
  pdl_wait();
  const int n = pt.n;
  const int c = blockIdx.y;
  const int r = next_client(c, n);
  int j = c + 1 - step;
  if (j < 0) j += n;
  if (j >= n) j -= n;
  const int64_t b = pt.begin(j), e = (j + 1 == n) ? pt.d : pt.begin(j + 1);
  const int64_t L = e - b;
  if (!(debug_ok(b <= e && e <= pt.d && pt.d <= out_ld, kDbgOutputRow) && debug_ok(r >= 0 && r < n, kDbgClient))) return;
  const float* src = out + (int64_t)c * out_ld + b;
  float* dst = out + (int64_t)r * out_ld + b;
  const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (VEC) {
    const int64_t i = t * 4;
    if (i + 4 <= L) {
      *reinterpret_cast<float4*>(dst + i) = *reinterpret_cast<const float4*>(src + i);
    } else {
      for (int64_t k = i; k < L; ++k) dst[k] = src[k];
    }
  } else {
    if (t < L) dst[t] = src[t];
  }
}

// ---------------------------------------------------------------------------
// Fused round: a CTA takes one tile of one sub-vector j and walks it through the
// ring in hop order -- client j, j+1, .., j+n-1 -- keeping the partial that
// would travel on the wire in registers.  The loads of the next UNR clients'
// rows are issued before the current ones are consumed (their addresses do not
// depend on data).  Only the partials of the last two hops are stored to the
// mailboxes: those are the only mailbox contents that survive a round in the
// hop-by-hop execution, so the final buffer state is the same.  The tile's
// consensus bits are staged in shared memory and written to all n output rows
// (what Share-Only leaves behind).
// ---------------------------------------------------------------------------
struct FusedArgs {
  Part pt;
  const float* U;
  int64_t ld;
  void* mail0;
  void* mail1;
  int64_t seg_pad;
  void* out;
  int64_t out_ld;
  int lam;      // consensus bit = (S > lam) | (S < lam_lo)
  int lam_lo;
  int zs;
  int mean;
  int tiles_per_seg;
  int64_t units;
  int owner_only;   // sign rules: write the consensus bits to the owner's row only (a share-only kernel follows)
};

template <typename P, int VPT, int UNR, bool ZS, int TPB>
__global__ void __launch_bounds__(TPB)
fused_sign_kernel(const FusedArgs a) {
  static_assert(VPT >= 1 && VPT <= 8, "tile width");
  constexpr int TILE = TPB * 4 * VPT;
  constexpr int WPT = (TPB / 8) * VPT;             // output words per tile
  __shared__ uint32_t sm_words[WPT];
  const Part pt = a.pt;
  const int n = pt.n;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const float* __restrict__ U = a.U;
  uint32_t* __restrict__ out = reinterpret_cast<uint32_t*>(a.out);

  for (int64_t u = blockIdx.x; u < a.units; u += gridDim.x) {
    const int j = (int)(u / a.tiles_per_seg);
    const int k = (int)(u % a.tiles_per_seg);
    const int64_t b = pt.begin(j), e = (j + 1 == n) ? pt.d : pt.begin(j + 1);
    const int64_t L = e - b;
    const int64_t t0 = (int64_t)k * TILE;
    if (t0 >= L) continue;
    if (!(debug_ok(b >= 0 && e <= pt.d && pt.d <= a.ld, kDbgUpdateRow) && debug_ok(L <= a.seg_pad, kDbgMailbox) &&
          debug_ok(j >= 0 && j < n, kDbgClient) && debug_ok(((e + 31) >> 5) <= a.out_ld, kDbgOutputRow)))
      continue;                                    // uniform over the CTA, like the test above                         // uniform over the CTA

    int64_t off[VPT];
    int nv[VPT];
    int acc[VPT][4];
#pragma unroll
    for (int v = 0; v < VPT; ++v) {
      off[v] = t0 + (int64_t)(v * TPB + tid) * 4;
      const int64_t rem = L - off[v];
      nv[v] = rem >= 4 ? 4 : (rem > 0 ? (int)rem : 0);
      acc[v][0] = acc[v][1] = acc[v][2] = acc[v][3] = 0;
    }
    const float* base = U + b;
    int c = j;
    for (int i0 = 0; i0 < n; i0 += UNR) {
      float4 x[UNR][VPT];
      int cc = c;
#pragma unroll
      for (int q = 0; q < UNR; ++q) {
        if (i0 + q < n) {
          const float* row = base + (int64_t)cc * a.ld;
#pragma unroll
          for (int v = 0; v < VPT; ++v)
            x[q][v] = nv[v] > 0 ? ld_stream(row + off[v]) : make_float4(0.f, 0.f, 0.f, 0.f);
          cc = next_client(cc, n);
        }
      }
#pragma unroll
      for (int q = 0; q < UNR; ++q) {
        if (i0 + q < n) {
          const int i = i0 + q;
#pragma unroll
          for (int v = 0; v < VPT; ++v) {
            acc[v][0] += sgn1<ZS>(x[q][v].x, a.zs);
            acc[v][1] += sgn1<ZS>(x[q][v].y, a.zs);
            acc[v][2] += sgn1<ZS>(x[q][v].z, a.zs);
            acc[v][3] += sgn1<ZS>(x[q][v].w, a.zs);
          }
          if (i >= 1 && i >= n - 2) {              // hop s = i-1 lands in client c's mailbox, set (s+1)&1
            P* m = reinterpret_cast<P*>((i & 1) ? a.mail1 : a.mail0) + (int64_t)c * a.seg_pad;
#pragma unroll
            for (int v = 0; v < VPT; ++v) {
              if (nv[v] == 4) {
                store4_stream(m + off[v], acc[v][0], acc[v][1], acc[v][2], acc[v][3]);
              } else {
#pragma unroll
                for (int q2 = 0; q2 < 3; ++q2)
                  if (q2 < nv[v]) m[off[v] + q2] = (P)acc[v][q2];
              }
            }
          }
          c = next_client(c, n);
        }
      }
    }

    // consensus bits: 4 per thread, 8 lanes make one word
#pragma unroll
    for (int v = 0; v < VPT; ++v) {
      uint32_t nib = 0;
#pragma unroll
      for (int q = 0; q < 4; ++q) nib |= (uint32_t)(q < nv[v] && ((acc[v][q] > a.lam) | (acc[v][q] < a.lam_lo))) << q;
      uint32_t word = nib << (4 * (lane & 7));
      word |= __shfl_xor_sync(0xffffffffu, word, 1);
      word |= __shfl_xor_sync(0xffffffffu, word, 2);
      word |= __shfl_xor_sync(0xffffffffu, word, 4);
      if ((lane & 7) == 0) sm_words[v * (TPB / 8) + warp * 4 + (lane >> 3)] = word;
    }
    __syncthreads();
    const int64_t left = L - t0;
    const int nw = left >= TILE ? WPT : (int)((left + 31) >> 5);
    const int64_t wb = (b + t0) >> 5;
    const int w = tid % WPT;
    if (w < nw) {
      const uint32_t val = sm_words[w];
      if (a.owner_only) {                            // client j-1 owns sub-vector j (Phase III is local to the owner)
        if (tid < WPT) out[(int64_t)(j == 0 ? n - 1 : j - 1) * a.out_ld + wb + w] = val;
      } else {
        for (int row = tid / WPT; row < n; row += TPB / WPT) out[(int64_t)row * a.out_ld + wb + w] = val;
      }
    }
    __syncthreads();
  }
}

template <int VPT, int UNR>
__global__ void __launch_bounds__(256)
fused_sum_kernel(const FusedArgs a) {
  constexpr int TILE = 256 * 4 * VPT;
  const Part pt = a.pt;
  const int n = pt.n;
  const int tid = threadIdx.x;
  const float* __restrict__ U = a.U;
  float* __restrict__ out = reinterpret_cast<float*>(a.out);
  const float fn = (float)n;

  for (int64_t u = blockIdx.x; u < a.units; u += gridDim.x) {
    const int j = (int)(u / a.tiles_per_seg);
    const int k = (int)(u % a.tiles_per_seg);
    const int64_t b = pt.begin(j), e = (j + 1 == n) ? pt.d : pt.begin(j + 1);
    const int64_t L = e - b;
    const int64_t t0 = (int64_t)k * TILE;
    if (t0 >= L) continue;
    if (!(debug_ok(b >= 0 && e <= pt.d && pt.d <= a.ld, kDbgUpdateRow) && debug_ok(L <= a.seg_pad, kDbgMailbox) &&
          debug_ok(j >= 0 && j < n, kDbgClient) && debug_ok(pt.d <= a.out_ld, kDbgOutputRow)))
      continue;                                    // uniform over the CTA, like the test above

    int64_t off[VPT];
    int nv[VPT];
    float acc[VPT][4];
#pragma unroll
    for (int v = 0; v < VPT; ++v) {
      off[v] = t0 + (int64_t)(v * 256 + tid) * 4;
      const int64_t rem = L - off[v];
      nv[v] = rem >= 4 ? 4 : (rem > 0 ? (int)rem : 0);
      acc[v][0] = acc[v][1] = acc[v][2] = acc[v][3] = 0.f;
    }
    const float* base = U + b;
    int c = j;
    for (int i0 = 0; i0 < n; i0 += UNR) {
      float4 x[UNR][VPT];
      int cc = c;
#pragma unroll
      for (int q = 0; q < UNR; ++q) {
        if (i0 + q < n) {
          const float* row = base + (int64_t)cc * a.ld;
#pragma unroll
          for (int v = 0; v < VPT; ++v)
            x[q][v] = nv[v] > 0 ? ld_stream(row + off[v]) : make_float4(0.f, 0.f, 0.f, 0.f);
          cc = next_client(cc, n);
        }
      }
#pragma unroll
      for (int q = 0; q < UNR; ++q) {
        if (i0 + q < n) {
          const int i = i0 + q;
#pragma unroll
          for (int v = 0; v < VPT; ++v) {
            if (i == 0) {                          // the sub-vector starts as client j's own values
              acc[v][0] = x[q][v].x; acc[v][1] = x[q][v].y; acc[v][2] = x[q][v].z; acc[v][3] = x[q][v].w;
            } else {                               // received partial + own, float32, ring order
              acc[v][0] = __fadd_rn(acc[v][0], x[q][v].x);
              acc[v][1] = __fadd_rn(acc[v][1], x[q][v].y);
              acc[v][2] = __fadd_rn(acc[v][2], x[q][v].z);
              acc[v][3] = __fadd_rn(acc[v][3], x[q][v].w);
            }
          }
          if (i >= 1 && i >= n - 2) {
            float* m = reinterpret_cast<float*>((i & 1) ? a.mail1 : a.mail0) + (int64_t)c * a.seg_pad;
#pragma unroll
            for (int v = 0; v < VPT; ++v) {
              if (nv[v] == 4) {
                *reinterpret_cast<float4*>(m + off[v]) = make_float4(acc[v][0], acc[v][1], acc[v][2], acc[v][3]);
              } else {
#pragma unroll
                for (int q2 = 0; q2 < 3; ++q2)
                  if (q2 < nv[v]) m[off[v] + q2] = acc[v][q2];
              }
            }
          }
          c = next_client(c, n);
        }
      }
    }
#pragma unroll
    for (int v = 0; v < VPT; ++v) {
      if (a.mean) {
#pragma unroll
        for (int q = 0; q < 4; ++q) acc[v][q] = __fdiv_rn(acc[v][q], fn);
      }
      float* dst = out + b + off[v];
      // owner_only: client j-1, the owner of sub-vector j, alone gets the result here (Phase III is local
      // to the owner); a share-only launch copies it to the other rows
      const int row0 = a.owner_only ? (j == 0 ? n - 1 : j - 1) : 0;
      const int row1 = a.owner_only ? row0 + 1 : n;
      if (nv[v] == 4) {
        const float4 val = make_float4(acc[v][0], acc[v][1], acc[v][2], acc[v][3]);
        for (int row = row0; row < row1; ++row) *reinterpret_cast<float4*>(dst + (int64_t)row * a.out_ld) = val;
      } else {
        for (int row = row0; row < row1; ++row) {
#pragma unroll
          for (int q = 0; q < 3; ++q)
            if (q < nv[v]) dst[(int64_t)row * a.out_ld + q] = acc[v][q];
        }
      }
    }
  }
}

// ---------------------------------------------------------------------------
// Model update that follows a round: each client applies the aggregate it holds
// to its own parameter row.  Sign rules (Appendix A, update rule): w <- w - eta*(+-1);
// plain ring-all-reduce (Section 2.2): w <- w - scale*sum with scale = eta/n.
// grid = (tiles over d, n clients); 4 coordinates per thread.
// ---------------------------------------------------------------------------
// VEC: 16-byte aligned rows; a thread then handles UPT float4 (one output word's worth of
// coordinates is 8 float4), all loaded before any is stored.
template <bool VEC, int UPT>
__global__ void __launch_bounds__(256)
apply_update_bits_kernel(const uint32_t* __restrict__ out, int64_t out_ld, float* __restrict__ Wt, int64_t ld_w,
                         int64_t d, float eta) {
  const int c = blockIdx.y;
  const int64_t k0 = ((int64_t)blockIdx.x * blockDim.x * UPT + threadIdx.x) * 4;
  float* wrow = Wt + (int64_t)c * ld_w;
  const uint32_t* orow = out + (int64_t)c * out_ld;
  float4 v[UPT];
  uint32_t nib[UPT];
#pragma unroll
  for (int u = 0; u < UPT; ++u) {
    const int64_t k = k0 + (int64_t)u * blockDim.x * 4;
    if (k < d) {
      nib[u] = (__ldg(orow + (k >> 5)) >> (int)(k & 31)) & 0xFu;
      if (VEC && k + 4 <= d) v[u] = *reinterpret_cast<float4*>(wrow + k);
    }
  }
#pragma unroll
  for (int u = 0; u < UPT; ++u) {
    const int64_t k = k0 + (int64_t)u * blockDim.x * 4;
    if (k >= d) continue;
    float* w = wrow + k;
    if (VEC && k + 4 <= d) {
      v[u].x = __fsub_rn(v[u].x, (nib[u] & 1u) ? eta : -eta);
      v[u].y = __fsub_rn(v[u].y, (nib[u] & 2u) ? eta : -eta);
      v[u].z = __fsub_rn(v[u].z, (nib[u] & 4u) ? eta : -eta);
      v[u].w = __fsub_rn(v[u].w, (nib[u] & 8u) ? eta : -eta);
      *reinterpret_cast<float4*>(w) = v[u];
    } else {
      for (int q = 0; q < 4 && k + q < d; ++q) w[q] = __fsub_rn(w[q], ((nib[u] >> q) & 1u) ? eta : -eta);
    }
  }
}

template <bool VEC, int UPT>
__global__ void __launch_bounds__(256)
apply_update_f32_kernel(const float* __restrict__ out, int64_t out_ld, float* __restrict__ Wt, int64_t ld_w,
                        int64_t d, float scale) {
  const int c = blockIdx.y;
  const int64_t k0 = ((int64_t)blockIdx.x * blockDim.x * UPT + threadIdx.x) * 4;
  float* wrow = Wt + (int64_t)c * ld_w;
  const float* grow = out + (int64_t)c * out_ld;
  float4 v[UPT], a[UPT];
#pragma unroll
  for (int u = 0; u < UPT; ++u) {
    const int64_t k = k0 + (int64_t)u * blockDim.x * 4;
    if (VEC && k + 4 <= d) {
      a[u] = ld_stream(grow + k);
      v[u] = *reinterpret_cast<float4*>(wrow + k);
    }
  }
#pragma unroll
  for (int u = 0; u < UPT; ++u) {
    const int64_t k = k0 + (int64_t)u * blockDim.x * 4;
    if (k >= d) continue;
    float* w = wrow + k;
    if (VEC && k + 4 <= d) {
      v[u].x = __fsub_rn(v[u].x, __fmul_rn(scale, a[u].x));
      v[u].y = __fsub_rn(v[u].y, __fmul_rn(scale, a[u].y));
      v[u].z = __fsub_rn(v[u].z, __fmul_rn(scale, a[u].z));
      v[u].w = __fsub_rn(v[u].w, __fmul_rn(scale, a[u].w));
      *reinterpret_cast<float4*>(w) = v[u];
    } else {
      const float* g = grow + k;
      for (int q = 0; q < 4 && k + q < d; ++q) w[q] = __fsub_rn(w[q], __fmul_rn(scale, g[q]));
    }
  }
}

// ---------------------------------------------------------------------------
// Phase I on its own (inspection / tests): int8 sign matrix.
// ---------------------------------------------------------------------------
template <bool ZS>
__global__ void __launch_bounds__(256)
quantize_kernel(const float* __restrict__ U, int64_t ld, int8_t* __restrict__ q, int64_t ld_q, int64_t d, int zs) {
  const int c = blockIdx.y;
  const int64_t k = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (k < d) q[(int64_t)c * ld_q + k] = (int8_t)sgn1<ZS>(U[(int64_t)c * ld + k], zs);
}

// ---------------------------------------------------------------------------
// Byzantine alterations (threat model of Section 3), applied before the ring.
// ids[0..f) are the Byzantine clients, ids[f..n) the honest ones in increasing id.
// ---------------------------------------------------------------------------
// kinds 1, 2, 5: element-wise, grid = (tiles over d, f Byzantine rows)
__global__ void __launch_bounds__(256)
inject_elementwise_kernel(int kind, const int* __restrict__ ids, const float* H, int64_t ld_h,
                          float* Uo, int64_t ld_u, const float* __restrict__ noise, int64_t ld_z,
                          const float* __restrict__ unif, int64_t ld_r, int64_t d, float scale, float sigma,
                          float prob) {
  const int bidx = blockIdx.y;
  const int id = ids[bidx];
  const int64_t k = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (k >= d) return;
  float v;
  if (kind == 1) {
    v = __fmul_rn(scale, H[(int64_t)id * ld_h + k]);
  } else if (kind == 2) {
    v = __fmul_rn(sigma, noise[(int64_t)bidx * ld_z + k]);
  } else {
    const float z = __fmul_rn(sigma, noise[(int64_t)bidx * ld_z + k]);
    v = (unif[(int64_t)bidx * ld_r + k] < prob) ? z : 0.0f;
  }
  Uo[(int64_t)id * ld_u + k] = v;
}

// kinds 3, 4: per-coordinate mean (and population std, two passes) over the
// honest rows in float64, rounded once to float32, written to every Byzantine row.
// No fused multiply-add anywhere: each operation rounds on its own.
template <int UNR>
__global__ void __launch_bounds__(256)
inject_stats_kernel(int kind, const int* __restrict__ ids, int f, int n, const float* H, int64_t ld_h,
                    float* Uo, int64_t ld_u, int64_t d, float scale, float kappa) {
  const int m = n - f;
  const int* good = ids + f;
  for (int64_t k = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; k < d; k += (int64_t)gridDim.x * blockDim.x) {
    double total = 0.0;
    for (int i0 = 0; i0 < m; i0 += UNR) {
      float x[UNR];
#pragma unroll
      for (int q = 0; q < UNR; ++q)
        if (i0 + q < m) x[q] = H[(int64_t)good[i0 + q] * ld_h + k];
#pragma unroll
      for (int q = 0; q < UNR; ++q)
        if (i0 + q < m) total = __dadd_rn(total, (double)x[q]);
    }
    const double mean = __ddiv_rn(total, (double)m);
    double vec;
    if (kind == 3) {
      vec = __dmul_rn((double)scale, mean);
    } else {
      double sq = 0.0;
      for (int i0 = 0; i0 < m; i0 += UNR) {
        float x[UNR];
#pragma unroll
        for (int q = 0; q < UNR; ++q)
          if (i0 + q < m) x[q] = H[(int64_t)good[i0 + q] * ld_h + k];
#pragma unroll
        for (int q = 0; q < UNR; ++q)
          if (i0 + q < m) {
            const double dev = __dsub_rn((double)x[q], mean);
            sq = __dadd_rn(sq, __dmul_rn(dev, dev));
          }
      }
      const double sd = __dsqrt_rn(__ddiv_rn(sq, (double)m));
      vec = __dsub_rn(mean, __dmul_rn((double)kappa, sd));
    }
    const float v = __double2float_rn(vec);
    for (int bq = 0; bq < f; ++bq) Uo[(int64_t)ids[bq] * ld_u + k] = v;
  }
}


// ---------------------------------------------------------------------------
// Random draws made inside the library.  The generator is counter-based, so a
// draw is a pure function of (seed, round, client, coordinate, stream) and no
// state travels between launches: Philox4x32 with 10 rounds (Salmon et al.,
// "Parallel random numbers: as easy as 1, 2, 3", SC'11), written here from its
// definition.  Four coordinates share one call: block q = k / 4 uses key
// (seed lo, seed hi) and counter (q lo, q hi, client, round * 256 + stream);
// word k % 4 belongs to coordinate k.
// ---------------------------------------------------------------------------
constexpr uint32_t kStreamUniform = 0;    // top 24 bits of the word, times 2^-24: uniform in [0, 1)
constexpr uint32_t kStreamNormal = 1;     // words (a, b) of a coordinate pair -> two normals (Box-Muller)

__device__ __forceinline__ uint4 philox4x32_10(uint4 c, uint2 key) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint32_t hi0 = __umulhi(0xD2511F53u, c.x), lo0 = 0xD2511F53u * c.x;
    const uint32_t hi1 = __umulhi(0xCD9E8D57u, c.z), lo1 = 0xCD9E8D57u * c.z;
    c = make_uint4(hi1 ^ c.y ^ key.x, lo1, hi0 ^ c.w ^ key.y, lo0);
    key.x += 0x9E3779B9u;
    key.y += 0xBB67AE85u;
  }
  return c;
}

__device__ __forceinline__ uint4 draw_block(uint64_t seed, uint32_t round, uint32_t client, uint32_t stream, int64_t q) {
  return philox4x32_10(make_uint4((uint32_t)q, (uint32_t)((uint64_t)q >> 32), client, round * 256u + stream),
                       make_uint2((uint32_t)seed, (uint32_t)(seed >> 32)));
}

__device__ __forceinline__ float uniform_from_word(uint32_t w) { return __fmul_rn((float)(w >> 8), 5.9604644775390625e-8f); }

// Box-Muller in float32: u1 = ((a >> 8) + 1) / 2^24 in (0, 1], u2 = (b >> 8) / 2^24;
// radius = sqrt(-2 ln u1); (radius cos 2 pi u2, radius sin 2 pi u2).
__device__ __forceinline__ void normal_pair(uint32_t a, uint32_t b, float& z0, float& z1) {
  const float u1 = __fmul_rn((float)((a >> 8) + 1u), 5.9604644775390625e-8f);
  const float two_u2 = __fmul_rn((float)(b >> 8), 1.1920928955078125e-7f);   // exact
  const float radius = __fsqrt_rn(__fmul_rn(-2.0f, logf(u1)));
  float s, c;
  sincospif(two_u2, &s, &c);
  z0 = __fmul_rn(radius, c);
  z1 = __fmul_rn(radius, s);
}

// Rows of raw draws, for inspection and as a building block of synthetic inputs:
// out[i][k] = mu + sigma * z (what = 1, standard normal z) or the uniform itself
// (what = 0).  Row i belongs to client first_client + i.  grid = (blocks of 4
// coordinates, rows).
__global__ void __launch_bounds__(256)
draw_matrix_kernel(int what, uint64_t seed, uint32_t round, int first_client, float* __restrict__ out, int64_t ld,
                   int64_t d, float mu, float sigma, int vec) {
  const int64_t q = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int64_t k = q * 4;
  if (k >= d) return;
  const uint32_t client = (uint32_t)(first_client + (int)blockIdx.y);
  float v[4];
  if (what == 0) {
    const uint4 w = draw_block(seed, round, client, kStreamUniform, q);
    v[0] = uniform_from_word(w.x); v[1] = uniform_from_word(w.y);
    v[2] = uniform_from_word(w.z); v[3] = uniform_from_word(w.w);
  } else {
    const uint4 w = draw_block(seed, round, client, kStreamNormal, q);
    normal_pair(w.x, w.y, v[0], v[1]);
    normal_pair(w.z, w.w, v[2], v[3]);
#pragma unroll
    for (int e = 0; e < 4; ++e) v[e] = __fadd_rn(mu, __fmul_rn(sigma, v[e]));
  }
  float* dst = out + (int64_t)blockIdx.y * ld + k;
  if (vec && k + 4 <= d) {
    *reinterpret_cast<float4*>(dst) = make_float4(v[0], v[1], v[2], v[3]);
  } else {
    for (int e = 0; e < 4 && k + e < d; ++e) dst[e] = v[e];
  }
}

// Alterations that consume randomness, drawing it here instead of reading
// pre-drawn matrices: kind 2 (b = sigma * z) and kind 5 (b = sigma * z where the
// coordinate's uniform is below prob, else 0).  Only the 4*f*d bytes of the
// Byzantine rows move.  For kind 5 the normals of a block are computed only if
// one of its four coordinates passes the test.  grid = (blocks of 4
// coordinates, f Byzantine rows).
__global__ void __launch_bounds__(256)
inject_generated_kernel(int kind, const int* __restrict__ ids, float* __restrict__ Uo, int64_t ld_u, int64_t d,
                        uint64_t seed, uint32_t round, float sigma, float prob, int vec) {
  const int64_t q = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int64_t k = q * 4;
  if (k >= d) return;
  const int id = ids[blockIdx.y];
  float v[4] = {0.f, 0.f, 0.f, 0.f};
  bool take[4] = {true, true, true, true};
  if (kind != 2) {
    const uint4 w = draw_block(seed, round, (uint32_t)id, kStreamUniform, q);
    take[0] = uniform_from_word(w.x) < prob; take[1] = uniform_from_word(w.y) < prob;
    take[2] = uniform_from_word(w.z) < prob; take[3] = uniform_from_word(w.w) < prob;
  }
  if (take[0] | take[1] | take[2] | take[3]) {
    const uint4 w = draw_block(seed, round, (uint32_t)id, kStreamNormal, q);
    float z[4];
    if (take[0] | take[1]) normal_pair(w.x, w.y, z[0], z[1]);
    if (take[2] | take[3]) normal_pair(w.z, w.w, z[2], z[3]);
#pragma unroll
    for (int e = 0; e < 4; ++e) v[e] = take[e] ? __fmul_rn(sigma, z[e]) : 0.0f;
  }
  float* dst = Uo + (int64_t)id * ld_u + k;
  if (vec && k + 4 <= d) {
    __stcs(reinterpret_cast<float4*>(dst), make_float4(v[0], v[1], v[2], v[3]));
  } else {
    for (int e = 0; e < 4 && k + e < d; ++e) dst[e] = v[e];
  }
}

// Kind 5 with the draws made here, for the usual case of a small prob: only the
// coordinates whose uniform passes the test need a normal, and the Box-Muller
// transform (log, square root, sine, cosine) costs several times what the
// uniform does.  A thread owns 8 coordinates (two uniform blocks).  The warp
// then compacts the coordinate pairs that need a normal into a list in shared
// memory (ballots give every pair its slot), works the list off 32 pairs at a
// time with all lanes busy -- the lane that handles a pair draws the pair's
// block of the normal stream and runs Box-Muller once -- and hands the values
// back through shared memory to the owners, which store two float4 each.
// Values and positions are those of inject_generated_kernel.  blockDim.x = 256;
// grid = (blocks of 2048 coordinates, f Byzantine rows).
__global__ void __launch_bounds__(256)
inject_sparse_generated_kernel(const int* __restrict__ ids, float* __restrict__ Uo, int64_t ld_u, int64_t d,
                               uint64_t seed, uint32_t round, float sigma, uint32_t thr, int vec) {
  __shared__ uint8_t sm_list[8][128];                // per warp: pairs that need a normal (lane * 4 + pair)
  __shared__ float2 sm_z[8][128];                    // per warp: the normals of those pairs
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;   // this thread owns coordinates 8t .. 8t+7
  const int64_t warp_t0 = t - lane;
  const uint32_t id = (uint32_t)ids[blockIdx.y];
  // uniforms: take[e] <=> (word >> 8) * 2^-24 < prob <=> (word >> 8) < thr, thr = ceil(prob * 2^24)
  uint32_t take = 0;
  if (t * 8 < d) {
    const uint4 w0 = draw_block(seed, round, id, kStreamUniform, 2 * t);
    const uint4 w1 = draw_block(seed, round, id, kStreamUniform, 2 * t + 1);
    take = (uint32_t)((w0.x >> 8) < thr) | (uint32_t)((w0.y >> 8) < thr) << 1 | (uint32_t)((w0.z >> 8) < thr) << 2 |
           (uint32_t)((w0.w >> 8) < thr) << 3 | (uint32_t)((w1.x >> 8) < thr) << 4 | (uint32_t)((w1.y >> 8) < thr) << 5 |
           (uint32_t)((w1.z >> 8) < thr) << 6 | (uint32_t)((w1.w >> 8) < thr) << 7;
  }
  // compaction: pair p of this lane gets slot (pairs of slots < p in the warp) + (lower lanes' pairs of slot p)
  int total = 0;
#pragma unroll
  for (int p = 0; p < 4; ++p) {
    const bool need = (take >> (2 * p)) & 3u;
    const uint32_t m = __ballot_sync(0xffffffffu, need);
    if (need) sm_list[warp][total + __popc(m & ((1u << lane) - 1u))] = (uint8_t)(lane * 4 + p);
    total += __popc(m);
  }
  __syncwarp();
  for (int i = lane; i < total; i += 32) {
    const int pid = sm_list[warp][i];
    const int owner = pid >> 2, p = pid & 3;
    // pair p of the owner covers coordinates 8 * (warp_t0 + owner) + 2p, +1: block 2 * (..) + p / 2 of the normal stream
    const uint4 w = draw_block(seed, round, id, kStreamNormal, 2 * (warp_t0 + owner) + (p >> 1));
    float z0, z1;
    if (p & 1) normal_pair(w.z, w.w, z0, z1);
    else normal_pair(w.x, w.y, z0, z1);
    sm_z[warp][pid] = make_float2(z0, z1);
  }
  __syncwarp();
  if (t * 8 >= d) return;
  float v[8];
#pragma unroll
  for (int p = 0; p < 4; ++p) {
    float2 z = make_float2(0.f, 0.f);
    if ((take >> (2 * p)) & 3u) z = sm_z[warp][lane * 4 + p];
    v[2 * p] = ((take >> (2 * p)) & 1u) ? __fmul_rn(sigma, z.x) : 0.0f;
    v[2 * p + 1] = ((take >> (2 * p + 1)) & 1u) ? __fmul_rn(sigma, z.y) : 0.0f;
  }
  const int64_t k = t * 8;
  float* dst = Uo + (int64_t)id * ld_u + k;
  if (vec && k + 8 <= d) {
    __stcs(reinterpret_cast<float4*>(dst), make_float4(v[0], v[1], v[2], v[3]));
    __stcs(reinterpret_cast<float4*>(dst) + 1, make_float4(v[4], v[5], v[6], v[7]));
  } else {
    for (int e = 0; e < 8 && k + e < d; ++e) dst[e] = v[e];
  }
}

// 128-bit variant of the element-wise alterations (rows 16-byte aligned).
__global__ void __launch_bounds__(256)
inject_elementwise_vec_kernel(int kind, const int* __restrict__ ids, const float* H, int64_t ld_h, float* Uo,
                              int64_t ld_u, const float* __restrict__ noise, int64_t ld_z,
                              const float* __restrict__ unif, int64_t ld_r, int64_t d, float scale, float sigma,
                              float prob) {
  const int bidx = blockIdx.y;
  const int id = ids[bidx];
  const int64_t k = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * 4;
  if (k >= d) return;
  float4 v;
  if (kind == 1) {
    const float4 h = *reinterpret_cast<const float4*>(H + (int64_t)id * ld_h + k);
    v = make_float4(__fmul_rn(scale, h.x), __fmul_rn(scale, h.y), __fmul_rn(scale, h.z), __fmul_rn(scale, h.w));
  } else {
    const float4 z = ld_stream(noise + (int64_t)bidx * ld_z + k);
    v = make_float4(__fmul_rn(sigma, z.x), __fmul_rn(sigma, z.y), __fmul_rn(sigma, z.z), __fmul_rn(sigma, z.w));
    if (kind != 2) {
      const float4 u = ld_stream(unif + (int64_t)bidx * ld_r + k);
      v.x = (u.x < prob) ? v.x : 0.0f;
      v.y = (u.y < prob) ? v.y : 0.0f;
      v.z = (u.z < prob) ? v.z : 0.0f;
      v.w = (u.w < prob) ? v.w : 0.0f;
    }
  }
  float* dst = Uo + (int64_t)id * ld_u + k;
  if (k + 4 <= d) {
    *reinterpret_cast<float4*>(dst) = v;
  } else {                                          // ragged end: never write past coordinate d-1
    const float t[4] = {v.x, v.y, v.z, v.w};
    for (int q = 0; k + q < d; ++q) dst[q] = t[q];
  }
}

// Mean / mean-shift alterations with the honest rows of a tile staged in shared
// memory by asynchronous 16-byte copies: the rows of the tile are requested far
// ahead of their use (many loads in flight without holding registers), the
// float64 sum consumes them eight rows at a time as they land, and the second
// pass (deviations) re-reads shared memory instead of HBM.  Each thread owns one
// float4 column of the tile, so no barrier is needed after the row offsets are
// published.  Arithmetic and order are those of inject_stats_kernel.
__device__ __forceinline__ void cp_async16(void* smem, const void* gmem) {
  const unsigned s = (unsigned)__cvta_generic_to_shared(smem);
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(s), "l"(gmem));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory"); }

template <int VW> struct StageVec;
template <> struct StageVec<1> { typedef float type; };
template <> struct StageVec<2> { typedef float2 type; };
template <> struct StageVec<4> { typedef float4 type; };

template <int VW>
__device__ __forceinline__ void cp_async_vw(void* smem, const void* gmem) {
  const unsigned s = (unsigned)__cvta_generic_to_shared(smem);
  if (VW == 4) asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(s), "l"(gmem));
  else if (VW == 2) asm volatile("cp.async.ca.shared.global [%0], [%1], 8;\n" ::"r"(s), "l"(gmem));
  else asm volatile("cp.async.ca.shared.global [%0], [%1], 4;\n" ::"r"(s), "l"(gmem));
}

// VW = floats per thread (1, 2 or 4): fewer floats per thread means more warps
// for the same shared-memory tile.
template <int VW, int DEPTH>
__global__ void inject_stats_smem_kernel(int kind, const int* __restrict__ ids, int f, int n, const float* H,
                                         int64_t ld_h, float* Uo, int64_t ld_u, int64_t d, float scale,
                                         float kappa) {
  constexpr int GROUP = 8;
  typedef typename StageVec<VW>::type V;
  extern __shared__ float4 sm_raw[];                // [mpad][blockDim.x] columns of V, then mpad row offsets
  V* sm_rows = reinterpret_cast<V*>(sm_raw);
  const int m = n - f;
  const int ngroups = (m + GROUP - 1) / GROUP;
  const int mpad = ngroups * GROUP;
  const int T = blockDim.x, tid = threadIdx.x;
  int64_t* rowoff = reinterpret_cast<int64_t*>(sm_rows + (size_t)mpad * T);
  for (int r = tid; r < mpad; r += T) rowoff[r] = (int64_t)ids[f + (r < m ? r : m - 1)] * ld_h;
  __syncthreads();
  const int64_t ntiles = (d + (int64_t)T * VW - 1) / ((int64_t)T * VW);
  V* col = sm_rows + tid;
  for (int64_t tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
    const int64_t k = (tile * T + tid) * VW;
    const bool active = k < d;
    const float* src = H + k;
    auto issue = [&](int g) {
      if (active && g < ngroups) {
#pragma unroll
        for (int q = 0; q < GROUP; ++q) {
          const int r = g * GROUP + q;
          if (r < m) cp_async_vw<VW>(col + (size_t)r * T, src + rowoff[r]);
        }
      }
      cp_async_commit();
    };
#pragma unroll 1
    for (int g = 0; g < DEPTH; ++g) issue(g);
    double tot[VW];
#pragma unroll
    for (int e = 0; e < VW; ++e) tot[e] = 0.0;
#pragma unroll 1
    for (int g = 0; g < ngroups; ++g) {
      cp_async_wait<DEPTH - 1>();
      if (active) {
        V x[GROUP];
#pragma unroll
        for (int q = 0; q < GROUP; ++q) x[q] = col[(size_t)(g * GROUP + q) * T];
#pragma unroll
        for (int q = 0; q < GROUP; ++q) {
          if (g * GROUP + q < m) {
            const float* xe = reinterpret_cast<const float*>(&x[q]);
#pragma unroll
            for (int e = 0; e < VW; ++e) tot[e] = __dadd_rn(tot[e], (double)xe[e]);
          }
        }
      }
      issue(g + DEPTH);
    }
    cp_async_wait<0>();
    if (!active) continue;
    double vec[VW];
    const double dm = (double)m;
    if (kind == 3) {
#pragma unroll
      for (int e = 0; e < VW; ++e) vec[e] = __dmul_rn((double)scale, __ddiv_rn(tot[e], dm));
    } else {
      double mean[VW], sq[VW];
#pragma unroll
      for (int e = 0; e < VW; ++e) { mean[e] = __ddiv_rn(tot[e], dm); sq[e] = 0.0; }
#pragma unroll 1
      for (int g = 0; g < ngroups; ++g) {
        V x[GROUP];
#pragma unroll
        for (int q = 0; q < GROUP; ++q) x[q] = col[(size_t)(g * GROUP + q) * T];
#pragma unroll
        for (int q = 0; q < GROUP; ++q) {
          if (g * GROUP + q < m) {
            const float* xe = reinterpret_cast<const float*>(&x[q]);
#pragma unroll
            for (int e = 0; e < VW; ++e) {
              const double dev = __dsub_rn((double)xe[e], mean[e]);
              sq[e] = __dadd_rn(sq[e], __dmul_rn(dev, dev));
            }
          }
        }
      }
#pragma unroll
      for (int e = 0; e < VW; ++e)
        vec[e] = __dsub_rn(mean[e], __dmul_rn((double)kappa, __dsqrt_rn(__ddiv_rn(sq[e], dm))));
    }
    float t[VW];
#pragma unroll
    for (int e = 0; e < VW; ++e) t[e] = __double2float_rn(vec[e]);
    if (k + VW <= d) {
      for (int bq = 0; bq < f; ++bq) *reinterpret_cast<V*>(Uo + (int64_t)ids[bq] * ld_u + k) = *reinterpret_cast<V*>(t);
    } else {
      for (int bq = 0; bq < f; ++bq)
        for (int e = 0; k + e < d; ++e) Uo[(int64_t)ids[bq] * ld_u + k + e] = t[e];
    }
  }
}

// Register-resident variant of the statistics kernel for up to 127 honest rows:
// a thread owns one coordinate, requests all of its honest values at once (they
// stay in registers), then runs the float64 sum and the float64 deviations over
// them -- the second pass costs no memory traffic at all.  MFULL rows are
// handled without predicates, up to MTAIL more with.
//
// The kernel is bound by instruction issue at low occupancy (the values of a
// coordinate fill most of a thread's registers), so what counts is instructions
// per element.  Two ways to address the rows:
//   STRIDED  honest rows are consecutive clients: row r is at base + r * stride,
//            one 32x32+64-bit multiply-add with r a constant; the Byzantine rows
//            are consecutive too and are stored by stepping a pointer;
//   table    row byte offsets travel as a kernel parameter (constant bank), the
//            Byzantine ids are read from the workspace.
struct HonestRows {
  int64_t byte_off[128];
};

// CTAs of 64 threads: the CTAs of one SM drift apart in phase (loading / computing) sooner than
// wider ones do, which keeps the memory pipe busier (n = 100, d = 25.6 M: 1.68 ms, against 1.71 ms
// with 128 threads, 1.73 ms with 32 and 1.81 ms with 256).
constexpr int kStatsThreads = 64;

__host__ __device__ constexpr int stats_min_blocks(int mfull) {
  return mfull <= 24 ? 8 : (mfull <= 40 ? 6 : (mfull <= 56 ? 5 : (mfull <= 80 ? 4 : (mfull <= 96 ? 3 : 2))));
}

template <int MFULL, int MTAIL, bool STRIDED>
__global__ void __launch_bounds__(kStatsThreads, stats_min_blocks(MFULL) * 128 / kStatsThreads)
inject_stats_reg_kernel(int kind, const __grid_constant__ HonestRows rows, uint32_t stride_bytes,
                        const int* __restrict__ ids, int f, int m, const float* H, float* Uo, int64_t ld_u, int64_t d,
                        float scale, float kappa) {
  const int64_t k = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (k >= d) return;
  // STRIDED: H points at the first honest row, Uo at the first Byzantine row
  const char* src = reinterpret_cast<const char*>(H + k);
  const int tail = m - MFULL;                        // 0..MTAIL rows beyond the unpredicated ones
  auto row_ptr = [&](int r) -> const float* {
    return reinterpret_cast<const float*>(STRIDED ? src + (uint64_t)stride_bytes * (uint32_t)r : src + rows.byte_off[r]);
  };
  float x[MFULL + MTAIL];
#pragma unroll
  for (int r = 0; r < MFULL; ++r) x[r] = __ldcs(row_ptr(r));
#pragma unroll
  for (int r = 0; r < MTAIL; ++r) {
    x[MFULL + r] = 0.0f;
    if (r < tail) x[MFULL + r] = __ldcs(row_ptr(MFULL + r));
  }
  double tot = 0.0;
#pragma unroll
  for (int r = 0; r < MFULL; ++r) tot = __dadd_rn(tot, (double)x[r]);
#pragma unroll
  for (int r = 0; r < MTAIL; ++r)
    if (r < tail) tot = __dadd_rn(tot, (double)x[MFULL + r]);
  const double dm = (double)m;
  const double mean = __ddiv_rn(tot, dm);
  double vec;
  if (kind == 3) {
    vec = __dmul_rn((double)scale, mean);
  } else {
    double sq = 0.0;
#pragma unroll
    for (int r = 0; r < MFULL; ++r) {
      asm volatile("" : "+f"(x[r]));                 // convert again rather than keep 2 registers per value
      const double dev = __dsub_rn((double)x[r], mean);
      sq = __dadd_rn(sq, __dmul_rn(dev, dev));
    }
#pragma unroll
    for (int r = 0; r < MTAIL; ++r) {
      if (r < tail) {
        asm volatile("" : "+f"(x[MFULL + r]));
        const double dev = __dsub_rn((double)x[MFULL + r], mean);
        sq = __dadd_rn(sq, __dmul_rn(dev, dev));
      }
    }
    vec = __dsub_rn(mean, __dmul_rn((double)kappa, __dsqrt_rn(__ddiv_rn(sq, dm))));
  }
  const float v = __double2float_rn(vec);
  if (STRIDED) {
    float* dst = Uo + k;
    for (int bq = 0; bq < f; ++bq, dst += ld_u) *dst = v;
  } else {
    for (int bq = 0; bq < f; ++bq) Uo[(int64_t)ids[bq] * ld_u + k] = v;
  }
}

// ---------------------------------------------------------------------------
// Coordinate-wise median / trimmed mean over the n client values of each
// coordinate (the server-side rules Section 5.1 compares against; they need all
// n slices at once, which is why they cannot run inside the ring, Section 3).
// A thread owns one coordinate: its n values are loaded into NB registers (n
// rounded up to a multiple of 8, the rest +Inf) and sorted by Batcher's odd-even
// merge sorting network, fully unrolled.  Every comparator of that network puts
// the smaller value at the lower index, so +Inf pads at the top never move and
// every comparator that would touch an index >= NB is left out at compile time:
// the network is the one for the next power of two restricted to indices < NB
// (1157 compare-exchanges for NB = 104 against 1792 for a 128-input bitonic
// network).  Arithmetic-bound: one min and one max per compare-exchange.
// ---------------------------------------------------------------------------
__host__ __device__ constexpr int pow2_at_least(int v) {
  int p = 1;
  while (p < v) p *= 2;
  return p;
}

#ifndef BRACE_STAT_TPB
#define BRACE_STAT_TPB 256
#endif
constexpr int kStatThreads = BRACE_STAT_TPB;

template <int NB>
__global__ void __launch_bounds__(kStatThreads)
coordinate_stat_kernel(int kind, int trim, int n, const float* __restrict__ U, int64_t ld, float* __restrict__ res,
                       int64_t d) {
  constexpr int NP = pow2_at_least(NB);
  const int64_t kc = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (kc >= d) return;
  const float* src = U + kc;
  float x[NB];
  // the host picks NB = n rounded up to a multiple of 8 (4 for n <= 4): only the last 7 (3) slots can be pads
  constexpr int SURE = NB > 8 ? NB - 7 : 1;
#pragma unroll
  for (int i = 0; i < NB; ++i) {
    if (i < SURE) x[i] = __ldcs(src + (int64_t)i * ld);
    else x[i] = (i < n) ? __ldcs(src + (int64_t)i * ld) : __int_as_float(0x7f800000);
  }
  // odd-even merge sort, ascending: merges of runs of length p, comparator distance k
#pragma unroll
  for (int p = 1; p < NP; p *= 2) {
#pragma unroll
    for (int k = p; k >= 1; k /= 2) {
#pragma unroll
      for (int i = 0; i < NB; ++i) {
        const int l = i + k;
        const int first = k % p;
        if (i >= first && ((i - first) % (2 * k)) < k && l < NB && (i / (2 * p)) == (l / (2 * p))) {
          const float lo = fminf(x[i], x[l]), hi = fmaxf(x[i], x[l]);
          x[i] = lo;
          x[l] = hi;
        }
      }
    }
  }
  float out;
  if (kind == 0) {                                   // median: middle value, or the mean of the two middle ones
    const int hi_idx = n >> 1, lo_idx = (n - 1) >> 1;
    float vlo = 0.f, vhi = 0.f;
    // n > NB - 8, so both middle positions lie in [(NB - 8) / 2, NB / 2]
#pragma unroll
    for (int i = (NB > 8 ? (NB - 8) / 2 : 0); i <= NB / 2 && i < NB; ++i) {
      if (i == lo_idx) vlo = x[i];
      if (i == hi_idx) vhi = x[i];
    }
    out = (lo_idx == hi_idx) ? vlo : __double2float_rn(__dmul_rn(0.5, __dadd_rn((double)vlo, (double)vhi)));
  } else {                                           // trimmed mean: drop `trim` smallest and largest, float64 mean
    double acc = 0.0;
#pragma unroll
    for (int i = 0; i < NB; ++i)
      if (i >= trim && i < n - trim) acc = __dadd_rn(acc, (double)x[i]);
    out = __double2float_rn(__ddiv_rn(acc, (double)(n - 2 * trim)));
  }
  res[kc] = out;
}

// ---------------------------------------------------------------------------
// Calibration: the rate at which this GPU executes the min/max operations the
// sorting network is made of, so that coordinate_stat_kernel can be held against
// a measured peak.  Every thread runs `iters` rounds of four stages of eight
// independent compare-exchanges on 16 registers (pair distances 1, 2, 4, 8, like
// the stages of a network): 64 min/max operations per round per thread, no
// memory traffic but one store at the end.
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
minmax_rate_kernel(float* __restrict__ out, int iters) {
  float x[16];
#pragma unroll
  for (int i = 0; i < 16; ++i) x[i] = (float)((threadIdx.x * 37 + i * 101 + blockIdx.x) % 251);
  for (int it = 0; it < iters; ++it) {
#pragma unroll
    for (int dist = 1; dist < 16; dist <<= 1) {
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        const int l = i ^ dist;
        if (l > i) {
          const float lo = fminf(x[i], x[l]), hi = fmaxf(x[i], x[l]);
          x[i] = hi;                                 // descending here, so that no stage finds its pairs in order
          x[l] = lo;
        }
      }
    }
    x[0] = -x[0];                                    // keep the data moving between rounds
  }
  float acc = 0.f;
#pragma unroll
  for (int i = 0; i < 16; ++i) acc += x[i];
  out[(int64_t)blockIdx.x * blockDim.x + threadIdx.x] = acc;
}

}  // namespace brace
