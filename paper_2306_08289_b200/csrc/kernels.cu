// Device kernels for sm_100a.
//
//   event kernel      a launch holds the items of one batch of worker-disjoint items (CTAs share out
//                     its (item, column tile) units round robin) or of several consecutive batches
//                     (column slices: every CTA owns a range of columns and walks all items in
//                     order). For a unit the item's rows (x, x~ of its two to four workers and the
//                     gradient rows it starts with) are read once with 256- or 128-bit loads, the
//                     item's operations are applied in registers in event order -- a gradient
//                     operation may fetch its worker's next gradient row -- and the state rows are
//                     written once. HBM-bound streaming work. Separate instances for two-, three- and
//                     four-worker items (the last with its rows as native 64-bit register pairs), for
//                     bf16 rows kept packed in registers, and for the dynamic without x~.
//   consensus kernel  per column: sum_i (x_i - xbar)^2 from shifted sums, fp64 across columns,
//                     warp shuffle + block reduce, per-block partials, fixed-order final sum.
//
// Per-element arithmetic (fp32, explicit FMAs, identical for fused and unfused schedules). Every
// stored value is updated as value + increment with ONE rounding at the value's own magnitude; the
// increment collects the mixing term and the jump and is itself small near consensus, so its
// rounding errors are small too:
//   gradient  dlt = x - x~;  tg = -gamma g;
//             x += fma(-c, dlt, tg);  x~ += fma(c, dlt, tg)            (Algorithm 1: matrix exponential, then
//                                                                       the two -gamma g lines; Eq. (dynamic), dN term)
//   comm      u_a = -c_a (x_a - x~_a);  u_b = -c_b (x_b - x~_b);         (mixing increments of x; those of x~ are -u)
//             m = (x_a - x_b) + (u_a - u_b)                             (x_a - x_b after both were mixed to t),
//             kept as an unevaluated sum m_hi + m_lo (error-free two-sums), because alpha~ can be
//             several times alpha and would amplify m's own rounding error into x~;
//             x_a += -alpha m + u_a;  x~_a += -alpha~ m - u_a;
//             x_b +=  alpha m + u_b;  x~_b +=  alpha~ m - u_b             (Eq. (dynamic), dM term)
//   (message-before-mix variant: m = x_a - x_b from the un-mixed rows.)
// The mixing coefficient c = -expm1(-2 eta (t - t_prev)) / 2 is evaluated in fp64 on the device
// from the event time and the worker's previous time carried by the descriptor, then rounded
// once to fp32.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdint>
#include <cstdlib>
#include <mutex>

#include "a2cid2_internal.h"

namespace a2 {

namespace {

constexpr int kThreads = 256;
#ifndef A2_EVENT_THREADS
#define A2_EVENT_THREADS 256
#endif
constexpr int kEventThreads = A2_EVENT_THREADS;  // threads per CTA of the event kernel

// ---------------------------------------------------------------------------------------------
// Vector access for the two storage types: BYTES = 32 (256-bit ld/st.global.v8, the widest
// sm_100 offers; needs 32-byte aligned rows) or 16 (128-bit, any row the ABI accepts).
// Vec<T, BYTES>::N elements per access; streaming (evict-first) cache policy on both sides.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void ld_u32x4(const void* p, uint32_t (&w)[4]) {
    const uint4 q = __ldcs(reinterpret_cast<const uint4*>(p));
    w[0] = q.x; w[1] = q.y; w[2] = q.z; w[3] = q.w;
}
__device__ __forceinline__ void st_u32x4(void* p, const uint32_t (&w)[4]) {
    __stcs(reinterpret_cast<uint4*>(p), make_uint4(w[0], w[1], w[2], w[3]));
}
__device__ __forceinline__ void ld_u32x8(const void* p, uint32_t (&w)[8]) {
    asm volatile("ld.global.cs.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]), "=r"(w[4]), "=r"(w[5]), "=r"(w[6]), "=r"(w[7])
                 : "l"(p));
}
__device__ __forceinline__ void st_u32x8(void* p, const uint32_t (&w)[8]) {
    asm volatile("st.global.cs.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                 :: "l"(p), "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]), "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7])
                 : "memory");
}

// Hint: bring the 128-byte line that holds p into L2 (no register, nothing to wait for).
__device__ __forceinline__ void prefetch_l2(const void* p) { asm volatile("prefetch.global.L2 [%0];" ::"l"(p)); }

template <int WORDS> struct Words;
template <> struct Words<4> {
    static __device__ __forceinline__ void ld(const void* p, uint32_t (&w)[4]) { ld_u32x4(p, w); }
    static __device__ __forceinline__ void st(void* p, const uint32_t (&w)[4]) { st_u32x4(p, w); }
};
template <> struct Words<8> {
    static __device__ __forceinline__ void ld(const void* p, uint32_t (&w)[8]) { ld_u32x8(p, w); }
    static __device__ __forceinline__ void st(void* p, const uint32_t (&w)[8]) { st_u32x8(p, w); }
};

template <typename T, int BYTES> struct Vec;

template <int BYTES> struct Vec<float, BYTES> {
    static constexpr int N = BYTES / 4;
    static __device__ __forceinline__ void load(const float* p, float (&v)[N]) {
        uint32_t w[N];
        Words<N>::ld(p, w);
#pragma unroll
        for (int k = 0; k < N; ++k) v[k] = __uint_as_float(w[k]);
    }
    static __device__ __forceinline__ void store(float* p, const float (&v)[N]) {
        uint32_t w[N];
#pragma unroll
        for (int k = 0; k < N; ++k) w[k] = __float_as_uint(v[k]);
        Words<N>::st(p, w);
    }
};

template <int BYTES> struct Vec<__nv_bfloat16, BYTES> {
    static constexpr int N = BYTES / 2;
    static __device__ __forceinline__ void load(const __nv_bfloat16* p, float (&v)[N]) {
        uint32_t w[N / 2];
        Words<N / 2>::ld(p, w);
#pragma unroll
        for (int k = 0; k < N / 2; ++k) {  // bf16 -> fp32 is a 16-bit shift
            v[2 * k] = __uint_as_float(w[k] << 16);
            v[2 * k + 1] = __uint_as_float(w[k] & 0xFFFF0000u);
        }
    }
    static __device__ __forceinline__ void store(__nv_bfloat16* p, const float (&v)[N]) {
        uint32_t w[N / 2];
#pragma unroll
        for (int k = 0; k < N / 2; ++k) {  // round to nearest even
            const __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * k], v[2 * k + 1]);
            w[k] = *reinterpret_cast<const uint32_t*>(&h);
        }
        Words<N / 2>::st(p, w);
    }
};

// Gradient event on one element: mixing over the elapsed time, then -gamma g on both buffers.
// ONE_ROUNDING (fp32 storage) adds mixing term and jump as a single increment; with bf16 storage the
// store's rounding dwarfs that refinement and the plain two-step form saves instructions.
template <bool ONE_ROUNDING>
__device__ __forceinline__ void grad_elem(float& x, float& xt, float c, float ngamma, float g) {
    const float dlt = __fsub_rn(x, xt);
    if (!ONE_ROUNDING) {
        x = __fmaf_rn(ngamma, g, __fmaf_rn(-c, dlt, x));
        xt = __fmaf_rn(ngamma, g, __fmaf_rn(c, dlt, xt));
        return;
    }
    const float tg = __fmul_rn(ngamma, g);
    x = __fadd_rn(x, __fmaf_rn(-c, dlt, tg));
    xt = __fadd_rn(xt, __fmaf_rn(c, dlt, tg));
}

// Communication event on one element of workers a and b. COMPENSATED carries the message as a
// two-term sum (fp32 storage); with bf16 storage the store's own rounding is five orders of
// magnitude larger than what the compensation recovers, so the plain difference is used.
template <bool COMPENSATED>
__device__ __forceinline__ void comm_elem(float& xa, float& xta, float& xb, float& xtb, float ca, float cb,
                                          float alpha, float alpha_t, bool msg_before_mix) {
    const float ua = __fmul_rn(-ca, __fsub_rn(xa, xta));
    const float ub = __fmul_rn(-cb, __fsub_rn(xb, xtb));
    if (!COMPENSATED) {  // plain two-step form: mix both workers, take the message, jump
        const float m_pre = __fsub_rn(xa, xb);
        xa = __fadd_rn(xa, ua);
        xta = __fsub_rn(xta, ua);
        xb = __fadd_rn(xb, ub);
        xtb = __fsub_rn(xtb, ub);
        const float m0 = msg_before_mix ? m_pre : __fsub_rn(xa, xb);
        xa = __fmaf_rn(-alpha, m0, xa);
        xta = __fmaf_rn(-alpha_t, m0, xta);
        xb = __fmaf_rn(alpha, m0, xb);
        xtb = __fmaf_rn(alpha_t, m0, xtb);
        return;
    }
    // raw + e_raw == x_a - x_b exactly (two-sum)
    const float nb = -xb;
    const float raw = __fadd_rn(xa, nb);
    float bv = __fsub_rn(raw, xa);
    float av = __fsub_rn(raw, bv);
    const float e_raw = __fadd_rn(__fsub_rn(xa, av), __fsub_rn(nb, bv));
    float m = raw, m_lo = e_raw;
    if (!msg_before_mix) {  // m + e_m == raw + du exactly
        const float du = __fsub_rn(ua, ub);
        m = __fadd_rn(raw, du);
        bv = __fsub_rn(m, raw);
        av = __fsub_rn(m, bv);
        m_lo = __fadd_rn(e_raw, __fadd_rn(__fsub_rn(raw, av), __fsub_rn(du, bv)));
    }
    xa = __fadd_rn(xa, __fmaf_rn(-alpha, m, __fmaf_rn(-alpha, m_lo, ua)));
    xta = __fadd_rn(xta, __fmaf_rn(-alpha_t, m, __fmaf_rn(-alpha_t, m_lo, -ua)));
    xb = __fadd_rn(xb, __fmaf_rn(alpha, m, __fmaf_rn(alpha, m_lo, ub)));
    xtb = __fadd_rn(xtb, __fmaf_rn(alpha_t, m, __fmaf_rn(alpha_t, m_lo, -ub)));
}

// ---------------------------------------------------------------------------------------------
// The same two updates on a PAIR of elements with sm_100's packed fp32 instructions (add/sub/mul/fma
// .rn.f32x2: two IEEE single-precision results per issued instruction, each rounded like the scalar
// form). The kernels with several events per row are short of issue slots, not of FP32 lanes; results
// are bit-identical to grad_elem / comm_elem (negations are moved, which round-to-nearest commutes with).
// ---------------------------------------------------------------------------------------------
#ifndef A2_F32X2_FP32
#define A2_F32X2_FP32 0  // fp32 rows: measured 1-3 % slower than the scalar forms (6.15 against 6.32 TB/s)
#endif
#ifndef A2_F32X2_FP32_KW4
#define A2_F32X2_FP32_KW4 1  // ... except in the four-worker instance with 256-bit accesses, which is short of issue
                             // slots: 37.4k -> 40.4k events/s (5.74 -> 6.25 TB/s) on the 64-worker ring
#endif
#ifndef A2_F32X2_BF16
#define A2_F32X2_BF16 1  // bf16 rows, whose kernels issue twice as much per byte: 1-2 % faster
#endif
using f32x2 = unsigned long long;
__device__ __forceinline__ f32x2 pk2(float lo, float hi) { f32x2 r; asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi)); return r; }
__device__ __forceinline__ void upk2(f32x2 v, float& lo, float& hi) { asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v)); }
__device__ __forceinline__ f32x2 add2(f32x2 a, f32x2 b) { f32x2 r; asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b)); return r; }
__device__ __forceinline__ f32x2 sub2(f32x2 a, f32x2 b) { f32x2 r; asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b)); return r; }
__device__ __forceinline__ f32x2 mul2(f32x2 a, f32x2 b) { f32x2 r; asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b)); return r; }
__device__ __forceinline__ f32x2 fma2(f32x2 a, f32x2 b, f32x2 c) { f32x2 r; asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c)); return r; }

struct GradK {  // per-operation constants of a gradient event, both lanes equal
    f32x2 c, nc, ngamma;
    __device__ __forceinline__ GradK(float c_, float ngamma_) : c(pk2(c_, c_)), nc(pk2(-c_, -c_)), ngamma(pk2(ngamma_, ngamma_)) {}
};
// The two updates on a native pair (one 64-bit register holding two fp32 columns).
template <bool ONE_ROUNDING>
__device__ __forceinline__ void grad_pair2(f32x2& x, f32x2& xt, const GradK& K, f32x2 g) {
    const f32x2 dlt = sub2(x, xt);
    if (!ONE_ROUNDING) {
        x = fma2(K.ngamma, g, fma2(K.nc, dlt, x));
        xt = fma2(K.ngamma, g, fma2(K.c, dlt, xt));
    } else {
        const f32x2 tg = mul2(K.ngamma, g);
        x = add2(x, fma2(K.nc, dlt, tg));
        xt = add2(xt, fma2(K.c, dlt, tg));
    }
}
template <bool ONE_ROUNDING>
__device__ __forceinline__ void grad_pair(float& x0, float& x1, float& xt0, float& xt1, const GradK& K, float g0, float g1) {
    f32x2 x = pk2(x0, x1), xt = pk2(xt0, xt1);
    grad_pair2<ONE_ROUNDING>(x, xt, K, pk2(g0, g1));
    upk2(x, x0, x1);
    upk2(xt, xt0, xt1);
}

struct CommK {  // per-operation constants of a communication event
    f32x2 nca, ncb, alpha, nalpha, alpha_t, nalpha_t;
    __device__ __forceinline__ CommK(float ca, float cb, float a, float at)
        : nca(pk2(-ca, -ca)), ncb(pk2(-cb, -cb)), alpha(pk2(a, a)), nalpha(pk2(-a, -a)), alpha_t(pk2(at, at)), nalpha_t(pk2(-at, -at)) {}
};
template <bool COMPENSATED>
__device__ __forceinline__ void comm_pair2(f32x2& xa, f32x2& xta, f32x2& xb, f32x2& xtb, const CommK& K, bool msg_before_mix) {
    const f32x2 ua = mul2(K.nca, sub2(xa, xta));
    const f32x2 ub = mul2(K.ncb, sub2(xb, xtb));
    if (!COMPENSATED) {
        const f32x2 m_pre = sub2(xa, xb);
        xa = add2(xa, ua);
        xta = sub2(xta, ua);
        xb = add2(xb, ub);
        xtb = sub2(xtb, ub);
        const f32x2 m0 = msg_before_mix ? m_pre : sub2(xa, xb);
        xa = fma2(K.nalpha, m0, xa);
        xta = fma2(K.nalpha_t, m0, xta);
        xb = fma2(K.alpha, m0, xb);
        xtb = fma2(K.alpha_t, m0, xtb);
    } else {
        const f32x2 raw = sub2(xa, xb);  // xa + (-xb)
        f32x2 bv = sub2(raw, xa);
        f32x2 av = sub2(raw, bv);
        const f32x2 e_raw = sub2(sub2(xa, av), add2(xb, bv));  // (xa - av) + (-xb - bv)
        f32x2 m = raw, m_lo = e_raw;
        if (!msg_before_mix) {
            const f32x2 du = sub2(ua, ub);
            m = add2(raw, du);
            bv = sub2(m, raw);
            av = sub2(m, bv);
            m_lo = add2(e_raw, add2(sub2(raw, av), sub2(du, bv)));
        }
        xa = add2(xa, fma2(K.nalpha, m, fma2(K.nalpha, m_lo, ua)));
        xta = sub2(xta, fma2(K.alpha_t, m, fma2(K.alpha_t, m_lo, ua)));     // + (-alpha~ m - alpha~ m_lo - ua)
        xb = add2(xb, fma2(K.alpha, m, fma2(K.alpha, m_lo, ub)));
        xtb = sub2(xtb, fma2(K.nalpha_t, m, fma2(K.nalpha_t, m_lo, ub)));  // + (alpha~ m + alpha~ m_lo - ub)
    }
}
template <bool COMPENSATED>
__device__ __forceinline__ void comm_pair(float& xa0, float& xa1, float& xta0, float& xta1, float& xb0, float& xb1,
                                          float& xtb0, float& xtb1, const CommK& K, bool msg_before_mix) {
    f32x2 xa = pk2(xa0, xa1), xta = pk2(xta0, xta1), xb = pk2(xb0, xb1), xtb = pk2(xtb0, xtb1);
    comm_pair2<COMPENSATED>(xa, xta, xb, xtb, K, msg_before_mix);
    upk2(xa, xa0, xa1);
    upk2(xta, xta0, xta1);
    upk2(xb, xb0, xb1);
    upk2(xtb, xtb0, xtb1);
}

// One operation on whole register rows of NE elements (NE even). PRECISE: the one-rounding / compensated forms
// (fp32 storage); PACKED: two elements per instruction.
template <bool PRECISE, bool PACKED, int NE>
__device__ __forceinline__ void grad_row(float (&x)[NE], float (&xt)[NE], float c, float ngamma, const float (&g)[NE]) {
    if constexpr (PACKED) {
        const GradK K(c, ngamma);
#pragma unroll
        for (int k = 0; k < NE; k += 2) grad_pair<PRECISE>(x[k], x[k + 1], xt[k], xt[k + 1], K, g[k], g[k + 1]);
    } else {
#pragma unroll
        for (int k = 0; k < NE; ++k) grad_elem<PRECISE>(x[k], xt[k], c, ngamma, g[k]);
    }
}
template <bool PRECISE, bool PACKED, int NE>
__device__ __forceinline__ void mix_row(float (&x)[NE], float (&xt)[NE], float c, float ngamma) {
    if constexpr (PACKED) {
        const GradK K(c, ngamma);
#pragma unroll
        for (int k = 0; k < NE; k += 2) grad_pair<PRECISE>(x[k], x[k + 1], xt[k], xt[k + 1], K, 0.f, 0.f);
    } else {
#pragma unroll
        for (int k = 0; k < NE; ++k) grad_elem<PRECISE>(x[k], xt[k], c, ngamma, 0.f);
    }
}
template <bool PRECISE, bool PACKED, int NE>
__device__ __forceinline__ void comm_row(float (&xa)[NE], float (&xta)[NE], float (&xb)[NE], float (&xtb)[NE], float ca, float cb,
                                         float alpha, float alpha_t, bool msg_before_mix) {
    if constexpr (PACKED) {
        const CommK K(ca, cb, alpha, alpha_t);
#pragma unroll
        for (int k = 0; k < NE; k += 2)
            comm_pair<PRECISE>(xa[k], xa[k + 1], xta[k], xta[k + 1], xb[k], xb[k + 1], xtb[k], xtb[k + 1], K, msg_before_mix);
    } else {
#pragma unroll
        for (int k = 0; k < NE; ++k) comm_elem<PRECISE>(xa[k], xta[k], xb[k], xtb[k], ca, cb, alpha, alpha_t, msg_before_mix);
    }
}

__device__ __forceinline__ double mix_coeff(double eta, double dt) { return -0.5 * expm1(-2.0 * eta * dt); }

// ---------------------------------------------------------------------------------------------
// Event kernel
// ---------------------------------------------------------------------------------------------
struct EventArgs {
    void* x;
    void* xt;
    const void* g;
    long long pitch;
    long long n_vec;  // vectors per row that hold at least one real column
    const DevItem* items;
    const DevOp* ops;
    int n_items;
    int n_ops;
    int n_tiles;
    double eta;
    float alpha, alpha_tilde, gamma;
    int msg_before_mix;
    int op_base;      // index, in the plan, of the launch's first operation (DevItem::op_first counts from the plan's)
    int slice_vec;    // column-slice launches: vectors of a row owned by one CTA (a multiple of 4); else 0
    int has_reloads;  // some operation of the launch fetches a gradient row in the middle of its item
};

// How a launch walks its (item, column tile) units.
//   round robin (SLICE = false)  one launch per batch of worker-disjoint items; unit u = (tile u / n_items, item
//       skewed by the tile index), CTA b takes units b, b + grid, ...: at any moment all CTAs stream through the
//       same few rows.
//   column slices (SLICE = true)  the launch's items may come from SEVERAL consecutive batches. CTA b owns the
//       vectors [b * slice_vec, (b + 1) * slice_vec) of every row and walks ALL items, in order, over that range
//       alone, the same thread always on the same columns. Every operation of the method is element-wise over
//       the parameter dimension (Eq. (dynamic) couples workers, never columns), so what an item needs from an
//       earlier item was written by the same thread: no grid-wide order is needed, hence no flag, no wait and
//       no launch boundary between batches. Every CTA does the same work, whatever the items cost.
template <bool SLICE, int TILE_VEC>
struct UnitWalk {
    long long v_lo, v_end;  // vectors of a row this CTA may touch
    int my_tiles, n_it;
    long long first, step, end;
    __device__ __forceinline__ UnitWalk(const EventArgs& p) {
        n_it = p.n_items;
        if (SLICE) {
            v_lo = (long long)blockIdx.x * p.slice_vec;
            v_end = v_lo + p.slice_vec < p.n_vec ? v_lo + p.slice_vec : p.n_vec;
            my_tiles = v_end > v_lo ? (int)((v_end - v_lo + TILE_VEC - 1) / TILE_VEC) : 0;
            first = 0; step = 1; end = (long long)n_it * my_tiles;
        } else {
            v_lo = 0; v_end = p.n_vec; my_tiles = p.n_tiles;
            first = blockIdx.x; step = gridDim.x; end = (long long)n_it * p.n_tiles;
        }
    }
    // unit -> item index and the first vector of the unit's tile
    __device__ __forceinline__ void map(long long unit, int& item_idx, long long& tile_v0) const {
        if (SLICE) {
            item_idx = (int)(unit / my_tiles);
            tile_v0 = v_lo + (unit % my_tiles) * (long long)TILE_VEC;
        } else {
            const int rem = (int)(unit % n_it);
            const long long tile = unit / n_it;
            const int skew = (int)((unsigned long long)tile % (unsigned)n_it);
            item_idx = rem + skew >= n_it ? rem + skew - n_it : rem + skew;
            tile_v0 = tile * (long long)TILE_VEC;
        }
    }
};

// KW = 2, 3 or 4: workers an item may hold (items of more than two workers come from A2_SCHED_CHAIN schedules).
// THREADS: threads per CTA (the four-worker instance trades threads for registers).
template <typename T, int BYTES, int UNROLL, int KW, int THREADS = kEventThreads, bool SLICE = false>
__global__ void __launch_bounds__(THREADS) k_apply_events(const EventArgs p) {
    using V = Vec<T, BYTES>;
    constexpr int N = V::N;
    __shared__ DevItem s_items[kMaxItemsPerLaunch];
    __shared__ float s_ca[kMaxOpsPerLaunch];
    __shared__ float s_cb[kMaxOpsPerLaunch];
    __shared__ unsigned char s_kind[kMaxOpsPerLaunch];
    __shared__ int s_reload[kMaxOpsPerLaunch];  // gradient row to fetch after a gradient operation, or -1

    for (int i = threadIdx.x; i < p.n_items; i += THREADS) s_items[i] = p.items[i];
    for (int o = threadIdx.x; o < p.n_ops; o += THREADS) {
        const DevOp op = p.ops[o];
        s_kind[o] = (unsigned char)op.kind;
        s_reload[o] = op.reload;
        const bool comm = op.kind == A2_OP_COMM || op.kind == A2_OP_COMM_AC || op.kind == A2_OP_COMM_BC ||
                          op.kind == A2_OP_COMM_AD || op.kind == A2_OP_COMM_BD || op.kind == A2_OP_COMM_CD;
        s_ca[o] = (float)mix_coeff(p.eta, op.t - op.t_prev_a);  // the operation's first (or only) worker
        s_cb[o] = comm ? (float)mix_coeff(p.eta, op.t - op.t_prev_b) : 0.f;
    }
    __syncthreads();

    T* const X = static_cast<T*>(p.x);
    T* const Xt = static_cast<T*>(p.xt);
    const T* const G = static_cast<const T*>(p.g);
    const float alpha = p.alpha, alpha_t = p.alpha_tilde, ngamma = -p.gamma;

    // unit -> (tile = unit / n_items, item = (unit % n_items + tile) % n_items). The skew by the tile index
    // makes every CTA walk through ALL items of the batch: without it a CTA whose stride shares a factor with
    // n_items would see only some of them, and items differ in cost (5 to 10 rows), which left the batches of
    // the 64-worker ring with a 2.7 % load imbalance across CTAs (0.4 % with the skew).
    // The bf16 kernel issues twice the instructions per byte and is helped by every instruction saved: it
    // advances (item, tile) incrementally and leaves absent rows uninitialised. The fp32 kernel measured about
    // 1 % FASTER with the 64-bit division per unit and the zero fill left in (6.37 against 6.30 TB/s on 64 rows
    // of 25.6e6 columns): it is bound by DRAM alone and the extra work between units spaces its bursts of loads;
    // so it keeps them.
    // (The three-worker instance issues more per byte and gains 3 % from leaving them out: 6.18 -> 6.38 TB/s.)
    constexpr bool kRecompute = sizeof(T) == 4 && KW == 2;
    const UnitWalk<SLICE, THREADS * UNROLL> walk(p);
    const long long v_end = walk.v_end;
    const int n_it = p.n_items;
    int rem = (int)(blockIdx.x % (unsigned)n_it);
    long long tile = blockIdx.x / (unsigned)n_it;
    int skew = (int)((unsigned long long)tile % (unsigned)n_it);
    const int step_rem = (int)(gridDim.x % (unsigned)n_it);
    const long long step_tile = gridDim.x / (unsigned)n_it;
    const int step_skew = (int)((unsigned long long)step_tile % (unsigned)n_it);
    for (long long unit = walk.first; unit < walk.end;
         unit += walk.step, rem += step_rem, tile += step_tile, skew += step_skew) {
        int item_idx;
        long long tile_v0;
        if (SLICE || kRecompute) {
            walk.map(unit, item_idx, tile_v0);
        } else {
            if (rem >= n_it) { rem -= n_it; tile += 1; skew += 1; }
            if (skew >= n_it) skew -= n_it;
            item_idx = rem + skew >= n_it ? rem + skew - n_it : rem + skew;
            tile_v0 = tile * (long long)(THREADS * UNROLL);
        }
        const DevItem it = s_items[item_idx];
        const long long v0 = tile_v0 + threadIdx.x;
        if (SLICE && tile_v0 + (long long)(threadIdx.x & ~31u) >= v_end) continue;  // nothing of this warp's is inside the slice
        const bool has_b = it.b >= 0, has_ga = it.slot_a >= 0, has_gb = it.slot_b >= 0;
        const bool has_c = KW >= 3 && it.c >= 0, has_gc = KW >= 3 && it.slot_c >= 0;
        const bool has_d = KW >= 4 && it.d >= 0, has_gd = KW >= 4 && it.slot_d >= 0;

        T* const pxa = X + (long long)it.a * p.pitch;
        T* const pxta = Xt + (long long)it.a * p.pitch;
        T* const pxb = X + (long long)(has_b ? it.b : it.a) * p.pitch;
        T* const pxtb = Xt + (long long)(has_b ? it.b : it.a) * p.pitch;
        T* const pxc = X + (long long)(has_c ? it.c : it.a) * p.pitch;
        T* const pxtc = Xt + (long long)(has_c ? it.c : it.a) * p.pitch;
        const T* const pga = G + (long long)(has_ga ? it.slot_a : 0) * p.pitch;
        const T* const pgb = G + (long long)(has_gb ? it.slot_b : 0) * p.pitch;
        const T* const pgc = G + (long long)(has_gc ? it.slot_c : 0) * p.pitch;
        T* const pxd = X + (long long)(has_d ? it.d : it.a) * p.pitch;
        T* const pxtd = Xt + (long long)(has_d ? it.d : it.a) * p.pitch;
        const T* const pgd = G + (long long)(has_gd ? it.slot_d : 0) * p.pitch;

        constexpr int UC = KW >= 3 ? UNROLL : 1, NC = KW >= 3 ? N : 1;  // no registers for a worker the instance never has
        constexpr int UD = KW >= 4 ? UNROLL : 1, ND = KW >= 4 ? N : 1;
        float xa[UNROLL][N], xta[UNROLL][N], xb[UNROLL][N], xtb[UNROLL][N], ga[UNROLL][N], gb[UNROLL][N];
        float xc[UC][NC], xtc[UC][NC], gc[UC][NC], xd[UD][ND], xtd[UD][ND], gd[UD][ND];
        bool live[UNROLL];
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            const long long v = v0 + (long long)u * THREADS;
            live[u] = v < v_end;
            const long long off = v * N;
            if (kRecompute) {
#pragma unroll
                for (int k = 0; k < N; ++k) { xb[u][k] = 0.f; xtb[u][k] = 0.f; ga[u][k] = 0.f; gb[u][k] = 0.f; xa[u][k] = 0.f; xta[u][k] = 0.f; }
                if constexpr (KW >= 3) {
#pragma unroll
                    for (int k = 0; k < NC; ++k) { xc[u][k] = 0.f; xtc[u][k] = 0.f; gc[u][k] = 0.f; }
                }
            }
            if (live[u]) {  // rows an item does not have are never read by its operations, nor stored
                V::load(pxa + off, xa[u]);
                V::load(pxta + off, xta[u]);
                if (has_b) {
                    V::load(pxb + off, xb[u]);
                    V::load(pxtb + off, xtb[u]);
                }
                if (has_ga) V::load(pga + off, ga[u]);
                if (has_gb) V::load(pgb + off, gb[u]);
                if constexpr (KW >= 3) {
                    if (has_c) {
                        V::load(pxc + off, xc[u]);
                        V::load(pxtc + off, xtc[u]);
                    }
                    if (has_gc) V::load(pgc + off, gc[u]);
                }
                if constexpr (KW >= 4) {
                    if (has_d) {
                        V::load(pxd + off, xd[u]);
                        V::load(pxtd + off, xtd[u]);
                    }
                    if (has_gd) V::load(pgd + off, gd[u]);
                }
            }
        }

        constexpr bool kPrecise = sizeof(T) == 4;
        constexpr bool kPacked = sizeof(T) == 4 ? ((KW >= 4 && BYTES == 32) ? (A2_F32X2_FP32_KW4 != 0) : (A2_F32X2_FP32 != 0))
                                                : (A2_F32X2_BF16 != 0);
        const bool before = p.msg_before_mix != 0;
        const int o_first = it.op_first - p.op_base;
        // Gradient rows that operations of this item fetch in the middle of the item (fresh gradients, Sec. 3.2) are
        // asked into L2 now, while the unit's own loads are in flight: the fetch then finds its line in L2 instead
        // of paying the DRAM and address-translation latency between two operations of the same worker. A hint
        // only: no register, nothing to wait for. (Asking the NEXT unit's rows into L2 the same way was measured
        // and dropped: no gain on any workload.)
        if (sizeof(T) == 4 && p.has_reloads) {  // (bf16 rows: items never change a worker's gradient row)
            for (int o = o_first; o < o_first + it.op_count; ++o) {
                const int rl = s_reload[o];
                if (rl >= 0) {
#pragma unroll
                    for (int u = 0; u < UNROLL; ++u)
                        if (live[u]) prefetch_l2(G + (long long)rl * p.pitch + (v0 + (long long)u * THREADS) * N);
                }
            }
        }
        for (int o = o_first; o < o_first + it.op_count; ++o) {
            const int kind = s_kind[o];
            const float ca = s_ca[o];
            // A gradient operation whose worker needs another row for its next one (fresh gradients, Sec. 3.2)
            // fetches it into the same registers as soon as it has used them: the load is in flight while the
            // item's following operations run.
            auto refetch = [&](auto& grow) {
                const int rl = s_reload[o];
                if (rl >= 0) {
                    const T* const pg = G + (long long)rl * p.pitch;
#pragma unroll
                    for (int u = 0; u < UNROLL; ++u)
                        if (live[u]) V::load(pg + (v0 + (long long)u * THREADS) * N, grow[u]);
                }
            };
            if (kind == A2_OP_GRAD_A) {
#pragma unroll
                for (int u = 0; u < UNROLL; ++u) grad_row<kPrecise, kPacked>(xa[u], xta[u], ca, ngamma, ga[u]);
                refetch(ga);
            } else if (kind == A2_OP_GRAD_B) {
#pragma unroll
                for (int u = 0; u < UNROLL; ++u) grad_row<kPrecise, kPacked>(xb[u], xtb[u], ca, ngamma, gb[u]);
                refetch(gb);
            } else if (kind == A2_OP_MIX_A) {  // mixing alone: a gradient event with a zero gradient
#pragma unroll
                for (int u = 0; u < UNROLL; ++u) mix_row<kPrecise, kPacked>(xa[u], xta[u], ca, ngamma);
            } else if (kind == A2_OP_COMM) {
                const float cb = s_cb[o];
#pragma unroll
                for (int u = 0; u < UNROLL; ++u) comm_row<kPrecise, kPacked>(xa[u], xta[u], xb[u], xtb[u], ca, cb, alpha, alpha_t, before);
            } else if constexpr (KW >= 3) {
                if (kind == A2_OP_GRAD_C) {
#pragma unroll
                    for (int u = 0; u < UNROLL; ++u) grad_row<kPrecise, kPacked>(xc[u], xtc[u], ca, ngamma, gc[u]);
                    refetch(gc);
                } else if (kind == A2_OP_COMM_AC) {
                    const float cb = s_cb[o];
#pragma unroll
                    for (int u = 0; u < UNROLL; ++u) comm_row<kPrecise, kPacked>(xa[u], xta[u], xc[u], xtc[u], ca, cb, alpha, alpha_t, before);
                } else if (kind == A2_OP_COMM_BC) {
                    const float cb = s_cb[o];
#pragma unroll
                    for (int u = 0; u < UNROLL; ++u) comm_row<kPrecise, kPacked>(xb[u], xtb[u], xc[u], xtc[u], ca, cb, alpha, alpha_t, before);
                } else if constexpr (KW >= 4) {
                    if (kind == A2_OP_GRAD_D) {
#pragma unroll
                        for (int u = 0; u < UNROLL; ++u) grad_row<kPrecise, kPacked>(xd[u], xtd[u], ca, ngamma, gd[u]);
                        refetch(gd);
                    } else {
                        const float cb = s_cb[o];
                        if (kind == A2_OP_COMM_AD) {
#pragma unroll
                            for (int u = 0; u < UNROLL; ++u) comm_row<kPrecise, kPacked>(xa[u], xta[u], xd[u], xtd[u], ca, cb, alpha, alpha_t, before);
                        } else if (kind == A2_OP_COMM_BD) {
#pragma unroll
                            for (int u = 0; u < UNROLL; ++u) comm_row<kPrecise, kPacked>(xb[u], xtb[u], xd[u], xtd[u], ca, cb, alpha, alpha_t, before);
                        } else {
#pragma unroll
                            for (int u = 0; u < UNROLL; ++u) comm_row<kPrecise, kPacked>(xc[u], xtc[u], xd[u], xtd[u], ca, cb, alpha, alpha_t, before);
                        }
                    }
                }
            }
        }

#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            const long long off = (v0 + (long long)u * THREADS) * N;
            if (live[u]) {
                V::store(pxa + off, xa[u]);
                V::store(pxta + off, xta[u]);
                if (has_b) {
                    V::store(pxb + off, xb[u]);
                    V::store(pxtb + off, xtb[u]);
                }
                if constexpr (KW >= 3) {
                    if (has_c) {
                        V::store(pxc + off, xc[u]);
                        V::store(pxtc + off, xtc[u]);
                    }
                }
                if constexpr (KW >= 4) {
                    if (has_d) {
                        V::store(pxd + off, xd[u]);
                        V::store(pxtd + off, xtd[u]);
                    }
                }
            }
        }
    }
}

// The two updates with x carried as an unevaluated sum x + xl inside an item (xl: what the roundings of x have lost
// so far; it starts at zero when the row is loaded and is added back, with one rounding, when the row is stored).
// xl enters the message, which alpha~ amplifies; the mixing difference x - x~ ignores it (c xl is second order:
// measured, the worst element of the 64-worker ring is the same with and without, and the kernel 3 % faster).
template <bool XLO>
__device__ __forceinline__ void grad_pair_x(f32x2& x, f32x2& xl, f32x2& xt, const GradK& K, f32x2 g) {
    const f32x2 dlt = sub2(x, xt);
    const f32x2 tg = mul2(K.ngamma, g);
    const f32x2 inc = fma2(K.nc, dlt, tg);
    const f32x2 s = add2(x, inc);
    if (XLO) xl = add2(xl, sub2(inc, sub2(s, x)));  // inc - (s - x): what the addition lost
    x = s;
    xt = add2(xt, fma2(K.c, dlt, tg));
}
template <bool XLO>
__device__ __forceinline__ void comm_pair_x(f32x2& xa, f32x2& xla, f32x2& xta, f32x2& xb, f32x2& xlb, f32x2& xtb, const CommK& K,
                                            bool msg_before_mix) {
    const f32x2 ua = mul2(K.nca, sub2(xa, xta));
    const f32x2 ub = mul2(K.ncb, sub2(xb, xtb));
    const f32x2 raw = sub2(xa, xb);
    f32x2 bv = sub2(raw, xa);
    f32x2 av = sub2(raw, bv);
    f32x2 e_raw = sub2(sub2(xa, av), add2(xb, bv));
    if (XLO) e_raw = add2(e_raw, sub2(xla, xlb));
    f32x2 m = raw, m_lo = e_raw;
    if (!msg_before_mix) {
        const f32x2 du = sub2(ua, ub);
        m = add2(raw, du);
        bv = sub2(m, raw);
        av = sub2(m, bv);
        m_lo = add2(e_raw, add2(sub2(raw, av), sub2(du, bv)));
    }
    const f32x2 ia = fma2(K.nalpha, m, fma2(K.nalpha, m_lo, ua));
    const f32x2 ib = fma2(K.alpha, m, fma2(K.alpha, m_lo, ub));
    const f32x2 sa = add2(xa, ia), sb = add2(xb, ib);
    if (XLO) {
        xla = add2(xla, sub2(ia, sub2(sa, xa)));
        xlb = add2(xlb, sub2(ib, sub2(sb, xb)));
    }
    xa = sa;
    xb = sb;
    xta = sub2(xta, fma2(K.alpha_t, m, fma2(K.alpha_t, m_lo, ua)));
    xtb = sub2(xtb, fma2(K.nalpha_t, m, fma2(K.nalpha_t, m_lo, ub)));
}

// ---------------------------------------------------------------------------------------------
// Four-worker items on fp32 rows with the rows held as NATIVE PAIRS: a row's 32 bytes arrive as four 64-bit
// registers (ld.global.cs.v4.b64), every operation is one of sm_100's packed fp32 instructions on such a register
// (add/sub/mul/fma.rn.f32x2: two IEEE results each, rounded like the scalar forms), and the row leaves as four
// 64-bit registers. k_apply_events reaches the same instructions from scalar registers through mov.b64 packs and
// unpacks around every operation; ncu showed those moves issuing about as many ALU instructions as there are
// packed FMA-pipe instructions, on a kernel that is short of issue slots (an item serves ten events, an SM holds
// only twelve of its warps). Per element the arithmetic, and so every bit of the result, is that of k_apply_events.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void ld_pairs(const float* p, f32x2 (&v)[4]) {
    asm volatile("ld.global.cs.v4.b64 {%0,%1,%2,%3}, [%4];" : "=l"(v[0]), "=l"(v[1]), "=l"(v[2]), "=l"(v[3]) : "l"(p));
}
__device__ __forceinline__ void st_pairs(float* p, const f32x2 (&v)[4]) {
    asm volatile("st.global.cs.v4.b64 [%0], {%1,%2,%3,%4};" ::"l"(p), "l"(v[0]), "l"(v[1]), "l"(v[2]), "l"(v[3]) : "memory");
}

// (Launch bounds without a minimum CTA count on purpose: ptxas then settles at 156-158 registers and two CTAs of
// 192 threads fit an SM. With an explicit minimum of one it takes more than 170, one CTA fits, and the kernel
// loses a third of its speed; with the registers capped at 128 for sixteen warps it gains nothing.)
// XLO: x is carried as the two-word value x + xl inside an item and rounded once, when the row is stored
// (A2_ROUND_PER_STORE); otherwise every event rounds x like every other value (A2_ROUND_PER_EVENT).
template <int KW, int THREADS, bool SLICE, bool XLO = false>
__global__ void __launch_bounds__(THREADS) k_apply_events_pairs(const EventArgs p) {
    constexpr int N = 8, NP = 4;  // fp32 columns and native pairs per 256-bit vector
    __shared__ DevItem s_items[kMaxItemsPerLaunch];
    __shared__ float s_ca[kMaxOpsPerLaunch];
    __shared__ float s_cb[kMaxOpsPerLaunch];
    __shared__ unsigned char s_kind[kMaxOpsPerLaunch];
    __shared__ int s_reload[kMaxOpsPerLaunch];

    for (int i = threadIdx.x; i < p.n_items; i += THREADS) s_items[i] = p.items[i];
    for (int o = threadIdx.x; o < p.n_ops; o += THREADS) {
        const DevOp op = p.ops[o];
        s_kind[o] = (unsigned char)op.kind;
        s_reload[o] = op.reload;
        const bool comm = op.kind == A2_OP_COMM || op.kind == A2_OP_COMM_AC || op.kind == A2_OP_COMM_BC ||
                          op.kind == A2_OP_COMM_AD || op.kind == A2_OP_COMM_BD || op.kind == A2_OP_COMM_CD;
        s_ca[o] = (float)mix_coeff(p.eta, op.t - op.t_prev_a);
        s_cb[o] = comm ? (float)mix_coeff(p.eta, op.t - op.t_prev_b) : 0.f;
    }
    __syncthreads();

    float* const X = static_cast<float*>(p.x);
    float* const Xt = static_cast<float*>(p.xt);
    const float* const G = static_cast<const float*>(p.g);
    const float alpha = p.alpha, alpha_t = p.alpha_tilde, ngamma = -p.gamma;
    const bool before = p.msg_before_mix != 0;

    const UnitWalk<SLICE, THREADS> walk(p);
    const long long v_end = walk.v_end;
    const int n_it = p.n_items;
    // (item, tile) of the round-robin walk advanced incrementally, as in k_apply_events
    int rem = (int)(blockIdx.x % (unsigned)n_it);
    long long tile = blockIdx.x / (unsigned)n_it;
    int skew = (int)((unsigned long long)tile % (unsigned)n_it);
    const int step_rem = (int)(gridDim.x % (unsigned)n_it);
    const long long step_tile = gridDim.x / (unsigned)n_it;
    const int step_skew = (int)((unsigned long long)step_tile % (unsigned)n_it);
    for (long long unit = walk.first; unit < walk.end; unit += walk.step, rem += step_rem, tile += step_tile, skew += step_skew) {
        int item_idx;
        long long tile_v0;
        if (SLICE) {
            walk.map(unit, item_idx, tile_v0);
        } else {
            if (rem >= n_it) { rem -= n_it; tile += 1; skew += 1; }
            if (skew >= n_it) skew -= n_it;
            item_idx = rem + skew >= n_it ? rem + skew - n_it : rem + skew;
            tile_v0 = tile * (long long)THREADS;
        }
        const DevItem it = s_items[item_idx];
        const long long v = tile_v0 + threadIdx.x;
        if (v >= v_end) continue;  // this thread's vector lies past the row (or past the slice)
        const long long off = v * N;
        const bool has_b = it.b >= 0, has_c = KW >= 3 && it.c >= 0, has_d = KW >= 4 && it.d >= 0;

        float* const pxa = X + (long long)it.a * p.pitch + off;
        float* const pxta = Xt + (long long)it.a * p.pitch + off;
        float* const pxb = X + (long long)(has_b ? it.b : it.a) * p.pitch + off;
        float* const pxtb = Xt + (long long)(has_b ? it.b : it.a) * p.pitch + off;
        float* const pxc = X + (long long)(has_c ? it.c : it.a) * p.pitch + off;
        float* const pxtc = Xt + (long long)(has_c ? it.c : it.a) * p.pitch + off;
        float* const pxd = X + (long long)(has_d ? it.d : it.a) * p.pitch + off;
        float* const pxtd = Xt + (long long)(has_d ? it.d : it.a) * p.pitch + off;

        constexpr int PC = KW >= 3 ? NP : 1, PD = KW >= 4 ? NP : 1;
        f32x2 xa[NP], xta[NP], xb[NP], xtb[NP], ga[NP], gb[NP], xc[PC], xtc[PC], gc[PC], xd[PD], xtd[PD], gd[PD];
        constexpr int LA = XLO ? NP : 1, LC = XLO ? PC : 1, LD = XLO ? PD : 1;
        f32x2 xla[LA], xlb[LA], xlc[LC], xld[LD];
        if (XLO) {
#pragma unroll
            for (int k = 0; k < LA; ++k) { xla[k] = 0ull; xlb[k] = 0ull; }
#pragma unroll
            for (int k = 0; k < LC; ++k) xlc[k] = 0ull;
#pragma unroll
            for (int k = 0; k < LD; ++k) xld[k] = 0ull;
        }
        ld_pairs(pxa, xa);
        ld_pairs(pxta, xta);
        if (has_b) {
            ld_pairs(pxb, xb);
            ld_pairs(pxtb, xtb);
        }
        if (it.slot_a >= 0) ld_pairs(G + (long long)it.slot_a * p.pitch + off, ga);
        if (it.slot_b >= 0) ld_pairs(G + (long long)it.slot_b * p.pitch + off, gb);
        if constexpr (KW >= 3) {
            if (has_c) {
                ld_pairs(pxc, xc);
                ld_pairs(pxtc, xtc);
            }
            if (it.slot_c >= 0) ld_pairs(G + (long long)it.slot_c * p.pitch + off, gc);
        }
        if constexpr (KW >= 4) {
            if (has_d) {
                ld_pairs(pxd, xd);
                ld_pairs(pxtd, xtd);
            }
            if (it.slot_d >= 0) ld_pairs(G + (long long)it.slot_d * p.pitch + off, gd);
        }

        const int o_first = it.op_first - p.op_base;
        if (p.has_reloads) {  // rows fetched in the middle of the item: asked into L2 now (see k_apply_events)
            for (int o = o_first; o < o_first + it.op_count; ++o) {
                const int rl = s_reload[o];
                if (rl >= 0) prefetch_l2(G + (long long)rl * p.pitch + off);
            }
        }
        for (int o = o_first; o < o_first + it.op_count; ++o) {
            const int kind = s_kind[o];
            const float ca = s_ca[o];
            auto grad = [&](f32x2 (&x)[NP], f32x2* xl, f32x2 (&xt)[NP], f32x2 (&g)[NP]) {
                const GradK K(ca, ngamma);
#pragma unroll
                for (int k = 0; k < NP; ++k) grad_pair_x<XLO>(x[k], xl[XLO ? k : 0], xt[k], K, g[k]);
                const int rl = s_reload[o];  // the worker's next gradient row, when it is another one
                if (rl >= 0) ld_pairs(G + (long long)rl * p.pitch + off, g);
            };
            auto comm = [&](f32x2 (&xp)[NP], f32x2* xlp, f32x2 (&xtp)[NP], f32x2 (&xq)[NP], f32x2* xlq, f32x2 (&xtq)[NP]) {
                const CommK K(ca, s_cb[o], alpha, alpha_t);
#pragma unroll
                for (int k = 0; k < NP; ++k)
                    comm_pair_x<XLO>(xp[k], xlp[XLO ? k : 0], xtp[k], xq[k], xlq[XLO ? k : 0], xtq[k], K, before);
            };
            if (kind == A2_OP_GRAD_A) {
                grad(xa, xla, xta, ga);
            } else if (kind == A2_OP_GRAD_B) {
                grad(xb, xlb, xtb, gb);
            } else if (kind == A2_OP_MIX_A) {  // mixing alone: a gradient event with a zero gradient
                const GradK K(ca, ngamma);
#pragma unroll
                for (int k = 0; k < NP; ++k) grad_pair_x<XLO>(xa[k], xla[XLO ? k : 0], xta[k], K, pk2(0.f, 0.f));
            } else if (kind == A2_OP_COMM) {
                comm(xa, xla, xta, xb, xlb, xtb);
            } else if constexpr (KW >= 3) {
                if (kind == A2_OP_GRAD_C) {
                    grad(xc, xlc, xtc, gc);
                } else if (kind == A2_OP_COMM_AC) {
                    comm(xa, xla, xta, xc, xlc, xtc);
                } else if (kind == A2_OP_COMM_BC) {
                    comm(xb, xlb, xtb, xc, xlc, xtc);
                } else if constexpr (KW >= 4) {
                    if (kind == A2_OP_GRAD_D) grad(xd, xld, xtd, gd);
                    else if (kind == A2_OP_COMM_AD) comm(xa, xla, xta, xd, xld, xtd);
                    else if (kind == A2_OP_COMM_BD) comm(xb, xlb, xtb, xd, xld, xtd);
                    else comm(xc, xlc, xtc, xd, xld, xtd);
                }
            }
        }

        if (XLO) {  // the row as stored: one rounding of x + xl
#pragma unroll
            for (int k = 0; k < NP; ++k) {
                xa[k] = add2(xa[k], xla[k]);
                if (has_b) xb[k] = add2(xb[k], xlb[k]);
                if (KW >= 3 && has_c) xc[k] = add2(xc[k], xlc[XLO && KW >= 3 ? k : 0]);
                if (KW >= 4 && has_d) xd[k] = add2(xd[k], xld[XLO && KW >= 4 ? k : 0]);
            }
        }

        st_pairs(pxa, xa);
        st_pairs(pxta, xta);
        if (has_b) {
            st_pairs(pxb, xb);
            st_pairs(pxtb, xtb);
        }
        if constexpr (KW >= 3) {
            if (has_c) {
                st_pairs(pxc, xc);
                st_pairs(pxtc, xtc);
            }
        }
        if constexpr (KW >= 4) {
            if (has_d) {
                st_pairs(pxd, xd);
                st_pairs(pxtd, xtd);
            }
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Event kernel of the dynamic without the momentum buffer (Eq. (baselinedynamic), Sec. 3.2):
//   gradient  x -= gamma g                       comm  m = x_a - x_b;  x_a -= alpha m;  x_b += alpha m
// Same descriptors, same unit mapping, half the rows: x_a, x_b and the gradient rows. There is no
// flow between events, so times play no part on the device and a mixing-only operation does nothing.
// ---------------------------------------------------------------------------------------------
#ifndef A2_PLAIN_UNROLL
#define A2_PLAIN_UNROLL 1  // 256-bit vectors per thread and tile
#endif
#ifndef A2_PLAIN_UNROLL_128
#define A2_PLAIN_UNROLL_128 2  // the same bytes per thread with 128-bit vectors
#endif
template <int BYTES> struct PlainCfg { static constexpr int UNROLL = BYTES == 32 ? A2_PLAIN_UNROLL : A2_PLAIN_UNROLL_128; };

template <typename T, int BYTES, int UNROLL, int KW, bool SLICE = false>
__global__ void __launch_bounds__(kEventThreads) k_apply_events_plain(const EventArgs p) {
    using V = Vec<T, BYTES>;
    constexpr int N = V::N;
    __shared__ DevItem s_items[kMaxItemsPerLaunch];
    __shared__ unsigned char s_kind[kMaxOpsPerLaunch];
    __shared__ int s_reload[kMaxOpsPerLaunch];
    for (int i = threadIdx.x; i < p.n_items; i += kEventThreads) s_items[i] = p.items[i];
    for (int o = threadIdx.x; o < p.n_ops; o += kEventThreads) {
        s_kind[o] = (unsigned char)p.ops[o].kind;
        s_reload[o] = p.ops[o].reload;
    }
    __syncthreads();

    T* const X = static_cast<T*>(p.x);
    const T* const G = static_cast<const T*>(p.g);
    const float alpha = p.alpha, ngamma = -p.gamma;
    const UnitWalk<SLICE, kEventThreads * UNROLL> walk(p);
    const long long v_end = walk.v_end;
    for (long long unit = walk.first; unit < walk.end; unit += walk.step) {
        int item_idx;
        long long tile_v0;
        walk.map(unit, item_idx, tile_v0);
        const DevItem it = s_items[item_idx];
        const bool has_b = it.b >= 0, has_ga = it.slot_a >= 0, has_gb = it.slot_b >= 0;
        const bool has_c = KW == 3 && it.c >= 0, has_gc = KW == 3 && it.slot_c >= 0;
        const long long v0 = tile_v0 + threadIdx.x;
        if (SLICE && tile_v0 + (long long)(threadIdx.x & ~31u) >= v_end) continue;
        T* const pxa = X + (long long)it.a * p.pitch;
        T* const pxb = X + (long long)(has_b ? it.b : it.a) * p.pitch;
        T* const pxc = X + (long long)(has_c ? it.c : it.a) * p.pitch;
        const T* const pga = G + (long long)(has_ga ? it.slot_a : 0) * p.pitch;
        const T* const pgb = G + (long long)(has_gb ? it.slot_b : 0) * p.pitch;
        const T* const pgc = G + (long long)(has_gc ? it.slot_c : 0) * p.pitch;

        constexpr int UC = KW == 3 ? UNROLL : 1, NC = KW == 3 ? N : 1;
        float xa[UNROLL][N], xb[UNROLL][N], ga[UNROLL][N], gb[UNROLL][N], xc[UC][NC], gc[UC][NC];
        bool live[UNROLL];
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            const long long v = v0 + (long long)u * kEventThreads;
            live[u] = v < v_end;
            const long long off = v * N;
#pragma unroll
            for (int k = 0; k < N; ++k) { xa[u][k] = 0.f; xb[u][k] = 0.f; ga[u][k] = 0.f; gb[u][k] = 0.f; }
            if constexpr (KW == 3) {
#pragma unroll
                for (int k = 0; k < NC; ++k) { xc[u][k] = 0.f; gc[u][k] = 0.f; }
            }
            if (live[u]) {
                V::load(pxa + off, xa[u]);
                if (has_b) V::load(pxb + off, xb[u]);
                if (has_ga) V::load(pga + off, ga[u]);
                if (has_gb) V::load(pgb + off, gb[u]);
                if constexpr (KW == 3) {
                    if (has_c) V::load(pxc + off, xc[u]);
                    if (has_gc) V::load(pgc + off, gc[u]);
                }
            }
        }
        bool dirty = false;
        const int o_first = it.op_first - p.op_base;
        if (p.has_reloads) {  // rows fetched in the middle of the item: asked into L2 now (see k_apply_events)
            for (int o = o_first; o < o_first + it.op_count; ++o) {
                const int rl = s_reload[o];
                if (rl >= 0) {
#pragma unroll
                    for (int u = 0; u < UNROLL; ++u)
                        if (live[u]) prefetch_l2(G + (long long)rl * p.pitch + (v0 + (long long)u * kEventThreads) * N);
                }
            }
        }
        for (int o = o_first; o < o_first + it.op_count; ++o) {
            const int kind = s_kind[o];
            if (kind == A2_OP_MIX_A) continue;
            dirty = true;
            auto refetch = [&](auto& grow) {  // the worker's next gradient row, when it is another one
                const int rl = s_reload[o];
                if (rl >= 0) {
                    const T* const pg = G + (long long)rl * p.pitch;
#pragma unroll
                    for (int u = 0; u < UNROLL; ++u)
                        if (live[u]) V::load(pg + (v0 + (long long)u * kEventThreads) * N, grow[u]);
                }
            };
            if (KW == 3 && (kind == A2_OP_GRAD_C || kind == A2_OP_COMM_AC || kind == A2_OP_COMM_BC)) {
#pragma unroll
                for (int u = 0; u < UC; ++u)
#pragma unroll
                    for (int k = 0; k < NC; ++k) {
                        if (kind == A2_OP_GRAD_C) {
                            xc[u][k] = __fmaf_rn(ngamma, gc[u][k], xc[u][k]);
                        } else if (kind == A2_OP_COMM_AC) {
                            const float m = __fsub_rn(xa[u][k], xc[u][k]);
                            xa[u][k] = __fmaf_rn(-alpha, m, xa[u][k]);
                            xc[u][k] = __fmaf_rn(alpha, m, xc[u][k]);
                        } else {
                            const float m = __fsub_rn(xb[u][k], xc[u][k]);
                            xb[u][k] = __fmaf_rn(-alpha, m, xb[u][k]);
                            xc[u][k] = __fmaf_rn(alpha, m, xc[u][k]);
                        }
                    }
                if constexpr (KW == 3) {
                    if (kind == A2_OP_GRAD_C) refetch(gc);
                }
                continue;
            }
#pragma unroll
            for (int u = 0; u < UNROLL; ++u)
#pragma unroll
                for (int k = 0; k < N; ++k) {
                    if (kind == A2_OP_GRAD_A) {
                        xa[u][k] = __fmaf_rn(ngamma, ga[u][k], xa[u][k]);
                    } else if (kind == A2_OP_GRAD_B) {
                        xb[u][k] = __fmaf_rn(ngamma, gb[u][k], xb[u][k]);
                    } else {
                        const float m = __fsub_rn(xa[u][k], xb[u][k]);
                        xa[u][k] = __fmaf_rn(-alpha, m, xa[u][k]);
                        xb[u][k] = __fmaf_rn(alpha, m, xb[u][k]);
                    }
                }
            if (kind == A2_OP_GRAD_A) refetch(ga);
            else if (kind == A2_OP_GRAD_B) refetch(gb);
        }
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            const long long off = (v0 + (long long)u * kEventThreads) * N;
            if (live[u] && dirty) {
                V::store(pxa + off, xa[u]);
                if (has_b) V::store(pxb + off, xb[u]);
                if constexpr (KW == 3) {
                    if (has_c) V::store(pxc + off, xc[u]);
                }
            }
        }
    }
}

// The same for bf16 rows. Half the bytes per column means twice the columns in flight for the same
// DRAM traffic, and widening every row to fp32 on arrival would spend the register file on that. So the
// rows stay packed (two columns per 32-bit register) while the loads are in flight, and each pair of
// columns is widened, taken through the item's operations and rounded back on its own.
#ifndef A2_PLAIN_BF16_UNROLL
#define A2_PLAIN_BF16_UNROLL 1  // 256-bit vectors per thread and tile (the 128-bit kernel takes twice as many)
#endif
#ifndef A2_PLAIN_BF16_GROUP
#define A2_PLAIN_BF16_GROUP 2
#endif

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }
__device__ __forceinline__ uint32_t bf16_pack(float lo, float hi) {  // round to nearest even
    const __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&h);
}

template <int WORDS, int UNROLL, int KW, bool SLICE = false>
__global__ void __launch_bounds__(kEventThreads) k_apply_events_plain_bf16(const EventArgs p) {
    __shared__ DevItem s_items[kMaxItemsPerLaunch];
    __shared__ unsigned char s_kind[kMaxOpsPerLaunch];
    for (int i = threadIdx.x; i < p.n_items; i += kEventThreads) s_items[i] = p.items[i];
    for (int o = threadIdx.x; o < p.n_ops; o += kEventThreads) s_kind[o] = (unsigned char)p.ops[o].kind;
    __syncthreads();

    __nv_bfloat16* const X = static_cast<__nv_bfloat16*>(p.x);
    const __nv_bfloat16* const G = static_cast<const __nv_bfloat16*>(p.g);
    const float alpha = p.alpha, ngamma = -p.gamma;
    const UnitWalk<SLICE, kEventThreads * UNROLL> walk(p);
    const long long v_end = walk.v_end;
    for (long long unit = walk.first; unit < walk.end; unit += walk.step) {
        int item_idx;
        long long tile_v0;
        walk.map(unit, item_idx, tile_v0);
        const DevItem it = s_items[item_idx];
        const bool has_b = it.b >= 0, has_ga = it.slot_a >= 0, has_gb = it.slot_b >= 0;
        const bool has_c = KW == 3 && it.c >= 0, has_gc = KW == 3 && it.slot_c >= 0;
        const long long v0 = tile_v0 + threadIdx.x;
        if (SLICE && tile_v0 + (long long)(threadIdx.x & ~31u) >= v_end) continue;
        __nv_bfloat16* const pxa = X + (long long)it.a * p.pitch;
        __nv_bfloat16* const pxb = X + (long long)(has_b ? it.b : it.a) * p.pitch;
        const __nv_bfloat16* const pga = G + (long long)(has_ga ? it.slot_a : 0) * p.pitch;
        const __nv_bfloat16* const pgb = G + (long long)(has_gb ? it.slot_b : 0) * p.pitch;
        __nv_bfloat16* const pxc = X + (long long)(has_c ? it.c : it.a) * p.pitch;
        const __nv_bfloat16* const pgc = G + (long long)(has_gc ? it.slot_c : 0) * p.pitch;
        constexpr int UC = KW == 3 ? UNROLL : 1, WC = KW == 3 ? WORDS : 1;
        uint32_t xc[UC][WC], gc[UC][WC];

        uint32_t xa[UNROLL][WORDS], xb[UNROLL][WORDS], ga[UNROLL][WORDS], gb[UNROLL][WORDS];
        bool live[UNROLL];
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            const long long v = v0 + (long long)u * kEventThreads;
            live[u] = v < v_end;
            const long long off = v * (2 * WORDS);
#pragma unroll
            for (int k = 0; k < WORDS; ++k) { xa[u][k] = 0u; xb[u][k] = 0u; ga[u][k] = 0u; gb[u][k] = 0u; }
            if constexpr (KW == 3) {
#pragma unroll
                for (int k = 0; k < WC; ++k) { xc[u][k] = 0u; gc[u][k] = 0u; }
                if (live[u]) {
                    if (has_c) Words<WORDS>::ld(pxc + off, xc[u]);
                    if (has_gc) Words<WORDS>::ld(pgc + off, gc[u]);
                }
            }
            if (live[u]) {
                Words<WORDS>::ld(pxa + off, xa[u]);
                if (has_b) Words<WORDS>::ld(pxb + off, xb[u]);
                if (has_ga) Words<WORDS>::ld(pga + off, ga[u]);
                if (has_gb) Words<WORDS>::ld(pgb + off, gb[u]);
            }
        }
        const int o_begin = it.op_first - p.op_base, o_end = o_begin + it.op_count;
        bool dirty = false;
        for (int o = o_begin; o < o_end; ++o) dirty |= s_kind[o] != A2_OP_MIX_A;
        constexpr int WG = A2_PLAIN_BF16_GROUP < WORDS ? A2_PLAIN_BF16_GROUP : WORDS;  // words widened and updated together
        constexpr int E = 2 * WG, EC = KW == 3 ? E : 1;
#pragma unroll
        for (int u = 0; u < UNROLL; ++u)
#pragma unroll
            for (int k0 = 0; k0 < WORDS; k0 += WG) {
                float a[E], b[E], fa[E], fb[E], c[EC], fc[EC];
#pragma unroll
                for (int w = 0; w < WG; ++w) {
                    a[2 * w] = bf16_lo(xa[u][k0 + w]); a[2 * w + 1] = bf16_hi(xa[u][k0 + w]);
                    b[2 * w] = bf16_lo(xb[u][k0 + w]); b[2 * w + 1] = bf16_hi(xb[u][k0 + w]);
                    fa[2 * w] = bf16_lo(ga[u][k0 + w]); fa[2 * w + 1] = bf16_hi(ga[u][k0 + w]);
                    fb[2 * w] = bf16_lo(gb[u][k0 + w]); fb[2 * w + 1] = bf16_hi(gb[u][k0 + w]);
                    if constexpr (KW == 3) {
                        c[2 * w] = bf16_lo(xc[u][k0 + w]); c[2 * w + 1] = bf16_hi(xc[u][k0 + w]);
                        fc[2 * w] = bf16_lo(gc[u][k0 + w]); fc[2 * w + 1] = bf16_hi(gc[u][k0 + w]);
                    }
                }
                for (int o = o_begin; o < o_end; ++o) {
                    const int kind = s_kind[o];
                    if (kind == A2_OP_GRAD_A) {
#pragma unroll
                        for (int e = 0; e < E; ++e) a[e] = __fmaf_rn(ngamma, fa[e], a[e]);
                    } else if (kind == A2_OP_GRAD_B) {
#pragma unroll
                        for (int e = 0; e < E; ++e) b[e] = __fmaf_rn(ngamma, fb[e], b[e]);
                    } else if (kind == A2_OP_COMM) {
#pragma unroll
                        for (int e = 0; e < E; ++e) {
                            const float m = __fsub_rn(a[e], b[e]);
                            a[e] = __fmaf_rn(-alpha, m, a[e]);
                            b[e] = __fmaf_rn(alpha, m, b[e]);
                        }
                    } else if (KW == 3 && kind == A2_OP_GRAD_C) {
#pragma unroll
                        for (int e = 0; e < EC; ++e) c[e] = __fmaf_rn(ngamma, fc[e], c[e]);
                    } else if (KW == 3 && kind == A2_OP_COMM_AC) {
#pragma unroll
                        for (int e = 0; e < EC; ++e) {
                            const float m = __fsub_rn(a[e], c[e]);
                            a[e] = __fmaf_rn(-alpha, m, a[e]);
                            c[e] = __fmaf_rn(alpha, m, c[e]);
                        }
                    } else if (KW == 3 && kind == A2_OP_COMM_BC) {
#pragma unroll
                        for (int e = 0; e < EC; ++e) {
                            const float m = __fsub_rn(b[e], c[e]);
                            b[e] = __fmaf_rn(-alpha, m, b[e]);
                            c[e] = __fmaf_rn(alpha, m, c[e]);
                        }
                    }
                }
#pragma unroll
                for (int w = 0; w < WG; ++w) {
                    xa[u][k0 + w] = bf16_pack(a[2 * w], a[2 * w + 1]);
                    xb[u][k0 + w] = bf16_pack(b[2 * w], b[2 * w + 1]);
                    if constexpr (KW == 3) xc[u][k0 + w] = bf16_pack(c[2 * w], c[2 * w + 1]);
                }
            }
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            const long long off = (v0 + (long long)u * kEventThreads) * (2 * WORDS);
            if (live[u] && dirty) {
                Words<WORDS>::st(pxa + off, xa[u]);
                if (has_b) Words<WORDS>::st(pxb + off, xb[u]);
                if constexpr (KW == 3) {
                    if (has_c) Words<WORDS>::st(pxc + off, xc[u]);
                }
            }
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Three-worker items on bf16 rows. Nine rows widened to fp32 take 126 registers and leave too few bytes in
// flight, so this instance keeps the rows packed (two columns per 32-bit register) while the loads are
// in flight and takes one pair of columns at a time through the item's operations: widen, apply every
// operation in order, round, pack. Per element the arithmetic is that of k_apply_events on bf16 rows.
// ---------------------------------------------------------------------------------------------
#ifndef A2_BF16_PACKED_GROUP
#define A2_BF16_PACKED_GROUP 2  // 32-bit words (pairs of columns) widened and updated together
#endif
template <int WORDS, int WG, bool SLICE = false>
__global__ void __launch_bounds__(kEventThreads) k_apply_events_bf16_packed(const EventArgs p) {
    __shared__ DevItem s_items[kMaxItemsPerLaunch];
    __shared__ float s_ca[kMaxOpsPerLaunch];
    __shared__ float s_cb[kMaxOpsPerLaunch];
    __shared__ unsigned char s_kind[kMaxOpsPerLaunch];
    for (int i = threadIdx.x; i < p.n_items; i += kEventThreads) s_items[i] = p.items[i];
    for (int o = threadIdx.x; o < p.n_ops; o += kEventThreads) {
        const DevOp op = p.ops[o];
        s_kind[o] = (unsigned char)op.kind;
        const bool comm = op.kind == A2_OP_COMM || op.kind == A2_OP_COMM_AC || op.kind == A2_OP_COMM_BC;
        s_ca[o] = (float)mix_coeff(p.eta, op.t - op.t_prev_a);
        s_cb[o] = comm ? (float)mix_coeff(p.eta, op.t - op.t_prev_b) : 0.f;
    }
    __syncthreads();

    __nv_bfloat16* const X = static_cast<__nv_bfloat16*>(p.x);
    __nv_bfloat16* const Xt = static_cast<__nv_bfloat16*>(p.xt);
    const __nv_bfloat16* const G = static_cast<const __nv_bfloat16*>(p.g);
    const float alpha = p.alpha, alpha_t = p.alpha_tilde, ngamma = -p.gamma;
    const bool before = p.msg_before_mix != 0;
    const UnitWalk<SLICE, kEventThreads> walk(p);
    for (long long unit = walk.first; unit < walk.end; unit += walk.step) {
        int item_idx;
        long long tile_v0;
        walk.map(unit, item_idx, tile_v0);
        const DevItem it = s_items[item_idx];
        const bool has_b = it.b >= 0, has_c = it.c >= 0;
        const bool has_ga = it.slot_a >= 0, has_gb = it.slot_b >= 0, has_gc = it.slot_c >= 0;
        const long long v = tile_v0 + threadIdx.x;
        if (v >= walk.v_end) continue;
        const long long off = v * (2 * WORDS);
        const long long ra = (long long)it.a * p.pitch + off;
        const long long rb = (long long)(has_b ? it.b : it.a) * p.pitch + off;
        const long long rc = (long long)(has_c ? it.c : it.a) * p.pitch + off;

        uint32_t xa[WORDS], xta[WORDS], xb[WORDS], xtb[WORDS], xc[WORDS], xtc[WORDS], ga[WORDS], gb[WORDS], gc[WORDS];
#pragma unroll
        for (int k = 0; k < WORDS; ++k) { xb[k] = 0u; xtb[k] = 0u; xc[k] = 0u; xtc[k] = 0u; ga[k] = 0u; gb[k] = 0u; gc[k] = 0u; }
        Words<WORDS>::ld(X + ra, xa);
        Words<WORDS>::ld(Xt + ra, xta);
        if (has_b) {
            Words<WORDS>::ld(X + rb, xb);
            Words<WORDS>::ld(Xt + rb, xtb);
        }
        if (has_c) {
            Words<WORDS>::ld(X + rc, xc);
            Words<WORDS>::ld(Xt + rc, xtc);
        }
        if (has_ga) Words<WORDS>::ld(G + (long long)it.slot_a * p.pitch + off, ga);
        if (has_gb) Words<WORDS>::ld(G + (long long)it.slot_b * p.pitch + off, gb);
        if (has_gc) Words<WORDS>::ld(G + (long long)it.slot_c * p.pitch + off, gc);

        const int o_begin = it.op_first - p.op_base, o_end = o_begin + it.op_count;
        constexpr int E = 2 * WG;  // columns taken through the operations together
#pragma unroll
        for (int k0 = 0; k0 < WORDS; k0 += WG) {
            float a[E], ta[E], b[E], tb[E], c[E], tc[E], fa[E], fb[E], fc[E];
#pragma unroll
            for (int w = 0; w < WG; ++w) {
                a[2 * w] = bf16_lo(xa[k0 + w]); a[2 * w + 1] = bf16_hi(xa[k0 + w]);
                ta[2 * w] = bf16_lo(xta[k0 + w]); ta[2 * w + 1] = bf16_hi(xta[k0 + w]);
                b[2 * w] = bf16_lo(xb[k0 + w]); b[2 * w + 1] = bf16_hi(xb[k0 + w]);
                tb[2 * w] = bf16_lo(xtb[k0 + w]); tb[2 * w + 1] = bf16_hi(xtb[k0 + w]);
                c[2 * w] = bf16_lo(xc[k0 + w]); c[2 * w + 1] = bf16_hi(xc[k0 + w]);
                tc[2 * w] = bf16_lo(xtc[k0 + w]); tc[2 * w + 1] = bf16_hi(xtc[k0 + w]);
                fa[2 * w] = bf16_lo(ga[k0 + w]); fa[2 * w + 1] = bf16_hi(ga[k0 + w]);
                fb[2 * w] = bf16_lo(gb[k0 + w]); fb[2 * w + 1] = bf16_hi(gb[k0 + w]);
                fc[2 * w] = bf16_lo(gc[k0 + w]); fc[2 * w + 1] = bf16_hi(gc[k0 + w]);
            }
            constexpr bool kPk = A2_F32X2_BF16 != 0;
            for (int o = o_begin; o < o_end; ++o) {
                const int kind = s_kind[o];
                const float ca = s_ca[o];
                if (kind == A2_OP_GRAD_A) {
                    grad_row<false, kPk>(a, ta, ca, ngamma, fa);
                } else if (kind == A2_OP_GRAD_B) {
                    grad_row<false, kPk>(b, tb, ca, ngamma, fb);
                } else if (kind == A2_OP_GRAD_C) {
                    grad_row<false, kPk>(c, tc, ca, ngamma, fc);
                } else if (kind == A2_OP_MIX_A) {
                    mix_row<false, kPk>(a, ta, ca, ngamma);
                } else {
                    const float cb = s_cb[o];
                    if (kind == A2_OP_COMM) comm_row<false, kPk>(a, ta, b, tb, ca, cb, alpha, alpha_t, before);
                    else if (kind == A2_OP_COMM_AC) comm_row<false, kPk>(a, ta, c, tc, ca, cb, alpha, alpha_t, before);
                    else comm_row<false, kPk>(b, tb, c, tc, ca, cb, alpha, alpha_t, before);
                }
            }
#pragma unroll
            for (int w = 0; w < WG; ++w) {
                xa[k0 + w] = bf16_pack(a[2 * w], a[2 * w + 1]); xta[k0 + w] = bf16_pack(ta[2 * w], ta[2 * w + 1]);
                xb[k0 + w] = bf16_pack(b[2 * w], b[2 * w + 1]); xtb[k0 + w] = bf16_pack(tb[2 * w], tb[2 * w + 1]);
                xc[k0 + w] = bf16_pack(c[2 * w], c[2 * w + 1]); xtc[k0 + w] = bf16_pack(tc[2 * w], tc[2 * w + 1]);
            }
        }
        Words<WORDS>::st(X + ra, xa);
        Words<WORDS>::st(Xt + ra, xta);
        if (has_b) {
            Words<WORDS>::st(X + rb, xb);
            Words<WORDS>::st(Xt + rb, xtb);
        }
        if (has_c) {
            Words<WORDS>::st(X + rc, xc);
            Words<WORDS>::st(Xt + rc, xtc);
        }
    }
}

// Vectors per thread and tile. 256-bit accesses: one vector per thread already keeps 4-6 rows x 32 B
// in flight per thread; 128-bit fp32 uses two.
template <typename T, int BYTES> struct EventCfg { static constexpr int UNROLL = 1; };
template <> struct EventCfg<float, 16> { static constexpr int UNROLL = 2; };

// ---------------------------------------------------------------------------------------------
// Consensus kernel
// ---------------------------------------------------------------------------------------------
template <typename T, int BYTES, bool FLUSH>
__global__ void __launch_bounds__(kThreads) k_consensus_partial(const T* __restrict__ X, const T* __restrict__ Xt,
                                                              long long pitch, int n, long long d, double eta,
                                                              const double* __restrict__ dt, double* __restrict__ partials) {
    using V = Vec<T, BYTES>;
    constexpr int N = V::N;
    extern __shared__ float s_c[];  // FLUSH: mixing coefficient of every worker to the common time
    __shared__ double s_warp[kThreads / 32];
    if (FLUSH) {
        for (int i = threadIdx.x; i < n; i += kThreads) s_c[i] = (float)mix_coeff(eta, dt[i]);
        __syncthreads();
    }
    const long long n_vec = (d + N - 1) / N;
    const double inv_n = 1.0 / (double)n;
    double acc = 0.0;
    for (long long v = (long long)blockIdx.x * kThreads + threadIdx.x; v < n_vec; v += (long long)gridDim.x * kThreads) {
        const long long off = v * N;
        float first[N], s1[N], s2[N];
        V::load(X + off, first);
        if (FLUSH) {
            float xt0[N];
            V::load(Xt + off, xt0);
            const float c = s_c[0];
#pragma unroll
            for (int k = 0; k < N; ++k) first[k] = __fmaf_rn(-c, __fsub_rn(first[k], xt0[k]), first[k]);
        }
#pragma unroll
        for (int k = 0; k < N; ++k) { s1[k] = 0.f; s2[k] = 0.f; }
#pragma unroll 4
        for (int i = 1; i < n; ++i) {
            float xi[N];
            V::load(X + (long long)i * pitch + off, xi);
            if (FLUSH) {
                float xti[N];
                V::load(Xt + (long long)i * pitch + off, xti);
                const float c = s_c[i];
#pragma unroll
                for (int k = 0; k < N; ++k) xi[k] = __fmaf_rn(-c, __fsub_rn(xi[k], xti[k]), xi[k]);
            }
#pragma unroll
            for (int k = 0; k < N; ++k) {
                const float s = __fsub_rn(xi[k], first[k]);  // shifted by the first row: no large cancellation later
                s1[k] += s;
                s2[k] = __fmaf_rn(s, s, s2[k]);
            }
        }
#pragma unroll
        for (int k = 0; k < N; ++k) {
            if (off + k < d) acc += (double)s2[k] - (double)s1[k] * (double)s1[k] * inv_n;
        }
    }
    // warp shuffle, then block reduce
#pragma unroll
    for (int s = 16; s > 0; s >>= 1) acc += __shfl_down_sync(0xffffffffu, acc, s);
    if ((threadIdx.x & 31) == 0) s_warp[threadIdx.x >> 5] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
        double tot = 0.0;
#pragma unroll
        for (int w = 0; w < kThreads / 32; ++w) tot += s_warp[w];
        partials[blockIdx.x] = tot;
    }
}

__global__ void __launch_bounds__(kThreads) k_consensus_final(const double* __restrict__ partials, int n_partials,
                                                            double* __restrict__ out) {
    __shared__ double s_warp[kThreads / 32];
    double acc = 0.0;
    for (int i = threadIdx.x; i < n_partials; i += kThreads) acc += partials[i];
#pragma unroll
    for (int s = 16; s > 0; s >>= 1) acc += __shfl_down_sync(0xffffffffu, acc, s);
    if ((threadIdx.x & 31) == 0) s_warp[threadIdx.x >> 5] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
        double tot = 0.0;
        for (int w = 0; w < kThreads / 32; ++w) tot += s_warp[w];
        out[0] = tot;
    }
}

#ifndef A2_EVENT4_THREADS
#define A2_EVENT4_THREADS 192  // threads per CTA of the four-worker instance
#endif
#ifndef A2_EVENT4_UNROLL_128
#define A2_EVENT4_UNROLL_128 2
#endif


// Grid of a launch. Round robin: one wave of resident CTAs (fewer if there are fewer units). Column slices: the same
// wave, each CTA owning `slice_vec` consecutive vectors of every row -- a multiple of 8 vectors (whole 128-byte
// lines) and at least one warp's worth, so that narrow rows give fewer, full warps instead of many empty ones.
struct GridShape {
    unsigned grid;
    int slice_vec;
};
inline GridShape grid_shape(bool slice, long long n_vec, long long n_units, long long wave) {
    GridShape g{0u, 0};
    if (!slice) {
        g.grid = (unsigned)(wave < n_units ? wave : n_units);
        return g;
    }
    long long per = (n_vec + wave - 1) / wave;
    per = (per + 7) / 8 * 8;
    if (per < 32) per = 32;
    if (per > 0x7FFFFFF8LL) per = 0x7FFFFFF8LL;
    g.slice_vec = (int)per;
    g.grid = (unsigned)((n_vec + per - 1) / per);
    return g;
}

template <typename T, int BYTES, int KW, int THREADS = kEventThreads, int U = EventCfg<T, BYTES>::UNROLL>
int launch_events_t(const EventLaunch& L, const DeviceInfo& dev, cudaStream_t stream) {
    constexpr int N = Vec<T, BYTES>::N;
    EventArgs a;
    a.x = L.x; a.xt = L.xt; a.g = L.g; a.pitch = L.pitch;
    a.n_vec = (L.d + N - 1) / N;
    a.items = L.items; a.ops = L.ops; a.n_items = L.n_items; a.n_ops = L.n_ops;
    const long long vec_per_tile = (long long)THREADS * U;
    a.n_tiles = (int)((a.n_vec + vec_per_tile - 1) / vec_per_tile);
    a.eta = L.eta; a.alpha = L.alpha; a.alpha_tilde = L.alpha_tilde; a.gamma = L.gamma;
    a.msg_before_mix = L.variant == A2_MSG_BEFORE_MIX;
    a.op_base = L.op_base;
    a.has_reloads = L.has_reloads ? 1 : 0;
    const long long n_units = (long long)a.n_items * a.n_tiles;
    const int per_sm = KW == 4 ? dev.event4_ctas_per_sm[BYTES == 32 ? 1 : 0]
                               : (KW == 3 ? dev.event3_ctas_per_sm : dev.event_ctas_per_sm)[L.dtype == A2_BF16 ? 1 : 0][BYTES == 32 ? 1 : 0];
    const GridShape gs = grid_shape(L.slice, a.n_vec, n_units, (long long)dev.sm_count * per_sm);
    a.slice_vec = gs.slice_vec;
    if (gs.grid < 1) return 0;
    if (L.slice) k_apply_events<T, BYTES, U, KW, THREADS, true><<<gs.grid, THREADS, 0, stream>>>(a);
    else k_apply_events<T, BYTES, U, KW, THREADS, false><<<gs.grid, THREADS, 0, stream>>>(a);
    return (int)cudaGetLastError();
}

int launch_events_pairs4(const EventLaunch& L, const DeviceInfo& dev, cudaStream_t stream) {
    constexpr int THREADS = A2_EVENT4_THREADS;
    EventArgs a;
    a.x = L.x; a.xt = L.xt; a.g = L.g; a.pitch = L.pitch;
    a.n_vec = (L.d + 7) / 8;
    a.items = L.items; a.ops = L.ops; a.n_items = L.n_items; a.n_ops = L.n_ops;
    a.n_tiles = (int)((a.n_vec + THREADS - 1) / THREADS);
    a.eta = L.eta; a.alpha = L.alpha; a.alpha_tilde = L.alpha_tilde; a.gamma = L.gamma;
    a.msg_before_mix = L.variant == A2_MSG_BEFORE_MIX;
    a.op_base = L.op_base;
    a.has_reloads = L.has_reloads ? 1 : 0;
    const long long n_units = (long long)a.n_items * a.n_tiles;
    const GridShape gs = grid_shape(L.slice, a.n_vec, n_units, (long long)dev.sm_count * dev.event4_ctas_per_sm[1]);
    a.slice_vec = gs.slice_vec;
    if (gs.grid < 1) return 0;
    if (L.round_per_store) {
        if (L.slice) k_apply_events_pairs<4, THREADS, true, true><<<gs.grid, THREADS, 0, stream>>>(a);
        else k_apply_events_pairs<4, THREADS, false, true><<<gs.grid, THREADS, 0, stream>>>(a);
    } else {
        if (L.slice) k_apply_events_pairs<4, THREADS, true><<<gs.grid, THREADS, 0, stream>>>(a);
        else k_apply_events_pairs<4, THREADS, false><<<gs.grid, THREADS, 0, stream>>>(a);
    }
    return (int)cudaGetLastError();
}

template <typename T, int BYTES, int KW>
int launch_plain_t(const EventLaunch& L, const DeviceInfo& dev, cudaStream_t stream) {
    constexpr int U = PlainCfg<BYTES>::UNROLL;
    constexpr int N = Vec<T, BYTES>::N;
    EventArgs a;
    a.x = L.x; a.xt = nullptr; a.g = L.g; a.pitch = L.pitch;
    a.n_vec = (L.d + N - 1) / N;
    a.items = L.items; a.ops = L.ops; a.n_items = L.n_items; a.n_ops = L.n_ops;
    const long long vec_per_tile = (long long)kEventThreads * U;
    a.n_tiles = (int)((a.n_vec + vec_per_tile - 1) / vec_per_tile);
    a.eta = 0.0; a.alpha = L.alpha; a.alpha_tilde = 0.f; a.gamma = L.gamma;
    a.msg_before_mix = 0;
    a.op_base = L.op_base;
    a.has_reloads = L.has_reloads ? 1 : 0;
    const long long n_units = (long long)a.n_items * a.n_tiles;
    const int per_sm = (KW == 3 ? dev.plain3_ctas_per_sm : dev.plain_ctas_per_sm)[L.dtype == A2_BF16 ? 1 : 0][BYTES == 32 ? 1 : 0];
    const GridShape gs = grid_shape(L.slice, a.n_vec, n_units, (long long)dev.sm_count * per_sm);
    a.slice_vec = gs.slice_vec;
    if (gs.grid < 1) return 0;
    if (L.slice) k_apply_events_plain<T, BYTES, U, KW, true><<<gs.grid, kEventThreads, 0, stream>>>(a);
    else k_apply_events_plain<T, BYTES, U, KW, false><<<gs.grid, kEventThreads, 0, stream>>>(a);
    return (int)cudaGetLastError();
}

template <int WORDS, int KW>
int launch_plain_bf16(const EventLaunch& L, const DeviceInfo& dev, cudaStream_t stream) {
    constexpr int U = A2_PLAIN_BF16_UNROLL * (8 / WORDS);
    EventArgs a;
    a.x = L.x; a.xt = nullptr; a.g = L.g; a.pitch = L.pitch;
    a.n_vec = (L.d + 2 * WORDS - 1) / (2 * WORDS);
    a.items = L.items; a.ops = L.ops; a.n_items = L.n_items; a.n_ops = L.n_ops;
    const long long vec_per_tile = (long long)kEventThreads * U;
    a.n_tiles = (int)((a.n_vec + vec_per_tile - 1) / vec_per_tile);
    a.eta = 0.0; a.alpha = L.alpha; a.alpha_tilde = 0.f; a.gamma = L.gamma;
    a.msg_before_mix = 0;
    a.op_base = L.op_base;
    a.has_reloads = L.has_reloads ? 1 : 0;
    const long long n_units = (long long)a.n_items * a.n_tiles;
    const long long wave = (long long)dev.sm_count * (KW == 3 ? dev.plain3_ctas_per_sm : dev.plain_ctas_per_sm)[1][WORDS == 8 ? 1 : 0];
    const GridShape gs = grid_shape(L.slice, a.n_vec, n_units, wave);
    a.slice_vec = gs.slice_vec;
    if (gs.grid < 1) return 0;
    if (L.slice) k_apply_events_plain_bf16<WORDS, U, KW, true><<<gs.grid, kEventThreads, 0, stream>>>(a);
    else k_apply_events_plain_bf16<WORDS, U, KW, false><<<gs.grid, kEventThreads, 0, stream>>>(a);
    return (int)cudaGetLastError();
}

// Resident CTAs per SM the persistent grid is sized for, measured on B200 with 64 rows of 25.6e6
// columns. fp32 rows, fused ring batches, 256-bit accesses: 1 CTA/SM 5.13 TB/s, 2: 6.33, 3: 6.01,
// 4: 5.97 -- beyond two CTAs the extra concurrent row streams cost more DRAM locality than the extra
// loads in flight buy. bf16 rows do twice the arithmetic per byte and want more warps: 128-bit
// accesses with 2 CTAs/SM 4.91 TB/s, 3: 5.81, 4: 5.84 (256-bit accesses, 127 registers: 5.45).
template <typename T> struct EventCtas { static constexpr int PER_SM = 2; };
template <> struct EventCtas<__nv_bfloat16> { static constexpr int PER_SM = 4; };

template <typename T, int BYTES, int KW>
cudaError_t event_occupancy(int* out) {
    int occ = 0;
    const cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(
        &occ, k_apply_events<T, BYTES, EventCfg<T, BYTES>::UNROLL, KW>, kEventThreads, 0);
    *out = occ > EventCtas<T>::PER_SM ? EventCtas<T>::PER_SM : (occ > 0 ? occ : 1);
    return e;
}

template <typename T, int BYTES, int KW>
cudaError_t plain_occupancy(int* out) {
    int occ = 0;
    const cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(
        &occ, k_apply_events_plain<T, BYTES, PlainCfg<BYTES>::UNROLL, KW>, kEventThreads, 0);
    // fp32 rows of 25.6e6 columns, one 256-bit vector per thread: two-worker items 2 CTAs/SM 5.65 TB/s, 3: 6.59,
    // 4: 6.18; three-worker items 2: 4.76, 3: 5.98, 4: 4.68 (two vectors per thread and 2 CTAs: 6.59 and 5.70)
    *out = occ > 3 ? 3 : (occ > 0 ? occ : 1);
    return e;
}

// 256-bit accesses are used for fp32 rows (bf16 rows are served better by 128-bit ones, see above) and
// need every row start on a 32-byte boundary.
bool rows_32B_aligned(const void* a, const void* b, const void* c, int64_t pitch, int32_t dtype) {
    if (dtype == A2_BF16) return false;
    static const bool force_narrow = a2::tuning_env("A2CID2_FORCE_128BIT") != nullptr;  // tuning override
    if (force_narrow) return false;
    const uintptr_t bits = reinterpret_cast<uintptr_t>(a) | reinterpret_cast<uintptr_t>(b) | reinterpret_cast<uintptr_t>(c);
    const int64_t pitch_bytes = pitch * (dtype == A2_BF16 ? 2 : 4);
    return (bits % 32 == 0) && (pitch_bytes % 32 == 0);
}

// Launches the partial-sum kernel with as many CTAs as are resident at once for this variant (at most
// `capacity`, the size of the scratch array) and returns that number: a grid of one full wave, so that no
// CTA waits for a slot while others already finish.
template <typename T, int BYTES, bool FLUSH>
int consensus_partial_variant(const T* X, const T* Xt, int64_t pitch, int32_t n, int64_t d, double eta, const double* dt,
                              double* partials, int capacity, int sm_count, cudaStream_t stream) {
    const size_t smem = FLUSH ? (size_t)n * sizeof(float) : 0;
    int occ = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, k_consensus_partial<T, BYTES, FLUSH>, kThreads, smem) != cudaSuccess || occ < 1)
        occ = 1;
    int grid = sm_count * occ;
    if (grid > capacity) grid = capacity;
    k_consensus_partial<T, BYTES, FLUSH><<<grid, kThreads, smem, stream>>>(X, Xt, pitch, n, d, eta, dt, partials);
    return grid;
}

template <typename T, int BYTES>
int launch_consensus_partial_t(const void* x, const void* xt, int64_t pitch, int32_t n, int64_t d, double eta,
                               const double* dt, double* partials, int capacity, int sm_count, cudaStream_t stream) {
    const T* X = static_cast<const T*>(x);
    const T* Xt = static_cast<const T*>(xt);
    if (dt) return consensus_partial_variant<T, BYTES, true>(X, Xt, pitch, n, d, eta, dt, partials, capacity, sm_count, stream);
    return consensus_partial_variant<T, BYTES, false>(X, Xt, pitch, n, d, eta, dt, partials, capacity, sm_count, stream);
}

}  // namespace

int query_device(DeviceInfo* info) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return (int)e;
    e = cudaDeviceGetAttribute(&info->sm_count, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return (int)e;
    if ((e = event_occupancy<float, 16, 2>(&info->event_ctas_per_sm[0][0])) != cudaSuccess) return (int)e;
    if ((e = event_occupancy<float, 32, 2>(&info->event_ctas_per_sm[0][1])) != cudaSuccess) return (int)e;
    if ((e = event_occupancy<__nv_bfloat16, 16, 2>(&info->event_ctas_per_sm[1][0])) != cudaSuccess) return (int)e;
    info->event_ctas_per_sm[1][1] = info->event_ctas_per_sm[1][0];
    {
        int occ = 0;
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(
            &occ, k_apply_events<float, 16, A2_EVENT4_UNROLL_128, 4, kEventThreads>, kEventThreads, 0);
        if (e != cudaSuccess) return (int)e;
        info->event4_ctas_per_sm[0] = occ > 2 ? 2 : (occ > 0 ? occ : 1);
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, k_apply_events_pairs<4, A2_EVENT4_THREADS, false>,
                                                          A2_EVENT4_THREADS, 0);
        if (e != cudaSuccess) return (int)e;
        info->event4_ctas_per_sm[1] = occ > 2 ? 2 : (occ > 0 ? occ : 1);
        if (const char* v = a2::tuning_env("A2CID2_EVENT4_CTAS_PER_SM")) {  // tuning override
            const int k = std::atoi(v);
            if (k > 0) info->event4_ctas_per_sm[0] = info->event4_ctas_per_sm[1] = k;
        }
    }
    if ((e = event_occupancy<float, 16, 3>(&info->event3_ctas_per_sm[0][0])) != cudaSuccess) return (int)e;
    if ((e = event_occupancy<float, 32, 3>(&info->event3_ctas_per_sm[0][1])) != cudaSuccess) return (int)e;
    {
        int occ = 0;
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, k_apply_events_bf16_packed<4, A2_BF16_PACKED_GROUP>, kEventThreads, 0);
        if (e != cudaSuccess) return (int)e;
        // measured on 64 bf16 rows of 25.6e6 columns, chained schedule: 128-bit accesses 2 CTAs/SM 5.02 TB/s, 3: 5.88,
        // 4: 4.99; 256-bit accesses 2: 6.05, 3: 5.47
        info->event3_ctas_per_sm[1][0] = occ > 3 ? 3 : (occ > 0 ? occ : 1);
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, k_apply_events_bf16_packed<8, A2_BF16_PACKED_GROUP>, kEventThreads, 0);
        if (e != cudaSuccess) return (int)e;
        info->event3_ctas_per_sm[1][1] = occ > 2 ? 2 : (occ > 0 ? occ : 1);
    }
    if ((e = plain_occupancy<float, 16, 2>(&info->plain_ctas_per_sm[0][0])) != cudaSuccess) return (int)e;
    if ((e = plain_occupancy<float, 32, 2>(&info->plain_ctas_per_sm[0][1])) != cudaSuccess) return (int)e;
    if ((e = plain_occupancy<float, 16, 3>(&info->plain3_ctas_per_sm[0][0])) != cudaSuccess) return (int)e;
    if ((e = plain_occupancy<float, 32, 3>(&info->plain3_ctas_per_sm[0][1])) != cudaSuccess) return (int)e;
    {
        int occ = 0;
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, k_apply_events_plain_bf16<4, 2 * A2_PLAIN_BF16_UNROLL, 2>,
                                                          kEventThreads, 0);
        if (e != cudaSuccess) return (int)e;
        info->plain_ctas_per_sm[1][0] = occ > 4 ? 4 : (occ > 0 ? occ : 1);
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, k_apply_events_plain_bf16<8, A2_PLAIN_BF16_UNROLL, 2>,
                                                          kEventThreads, 0);
        if (e != cudaSuccess) return (int)e;
        info->plain_ctas_per_sm[1][1] = occ > 4 ? 4 : (occ > 0 ? occ : 1);
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, k_apply_events_plain_bf16<4, 2 * A2_PLAIN_BF16_UNROLL, 3>,
                                                          kEventThreads, 0);
        if (e != cudaSuccess) return (int)e;
        info->plain3_ctas_per_sm[1][0] = occ > 3 ? 3 : (occ > 0 ? occ : 1);
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, k_apply_events_plain_bf16<8, A2_PLAIN_BF16_UNROLL, 3>,
                                                          kEventThreads, 0);
        if (e != cudaSuccess) return (int)e;
        // bf16 rows of 25.6e6 columns, 256-bit accesses, chained schedule: 2 CTAs/SM 5.37 TB/s, 3: 6.36, 4: 5.12
        info->plain3_ctas_per_sm[1][1] = occ > 3 ? 3 : (occ > 0 ? occ : 1);
    }
    if (const char* v = a2::tuning_env("A2CID2_PLAIN_CTAS_PER_SM")) {  // tuning override, as for the event kernel
        const int k = std::atoi(v);
        if (k > 0)
            for (auto& row : info->plain_ctas_per_sm)
                for (int& c : row) c = k;
    }
    if (const char* v = a2::tuning_env("A2CID2_PLAIN3_CTAS_PER_SM")) {  // the same for the three-worker instances
        const int k = std::atoi(v);
        if (k > 0)
            for (auto& row : info->plain3_ctas_per_sm)
                for (int& c : row) c = k;
    }
    info->consensus_ctas_per_sm = 8;  // capacity of the partial-sum scratch, CTAs per SM
    if (const char* v = a2::tuning_env("A2CID2_EVENT_CTAS_PER_SM")) {  // tuning override: resident CTAs per SM of the event kernel
        const int k = std::atoi(v);
        if (k > 0)
            for (auto& row : info->event_ctas_per_sm)
                for (int& c : row) c = k;
    }
    if (const char* v = a2::tuning_env("A2CID2_EVENT3_CTAS_PER_SM")) {  // the same for the three-worker instances
        const int k = std::atoi(v);
        if (k > 0)
            for (auto& row : info->event3_ctas_per_sm)
                for (int& c : row) c = k;
    }
    return 0;
}

template <int WORDS>
int launch_bf16_packed(const EventLaunch& L, const DeviceInfo& dev, cudaStream_t stream) {
    EventArgs a;
    a.x = L.x; a.xt = L.xt; a.g = L.g; a.pitch = L.pitch;
    a.n_vec = (L.d + 2 * WORDS - 1) / (2 * WORDS);
    a.items = L.items; a.ops = L.ops; a.n_items = L.n_items; a.n_ops = L.n_ops;
    a.n_tiles = (int)((a.n_vec + kEventThreads - 1) / kEventThreads);
    a.eta = L.eta; a.alpha = L.alpha; a.alpha_tilde = L.alpha_tilde; a.gamma = L.gamma;
    a.msg_before_mix = L.variant == A2_MSG_BEFORE_MIX;
    a.op_base = L.op_base;
    a.has_reloads = L.has_reloads ? 1 : 0;
    const long long n_units = (long long)a.n_items * a.n_tiles;
    const GridShape gs = grid_shape(L.slice, a.n_vec, n_units, (long long)dev.sm_count * dev.event3_ctas_per_sm[1][WORDS == 8 ? 1 : 0]);
    a.slice_vec = gs.slice_vec;
    if (gs.grid < 1) return 0;
    if (L.slice) k_apply_events_bf16_packed<WORDS, A2_BF16_PACKED_GROUP, true><<<gs.grid, kEventThreads, 0, stream>>>(a);
    else k_apply_events_bf16_packed<WORDS, A2_BF16_PACKED_GROUP, false><<<gs.grid, kEventThreads, 0, stream>>>(a);
    return (int)cudaGetLastError();
}

// Rows on 32-byte boundaries (what the 256-bit kernels, and with them A2_ROUND_PER_STORE, need).
bool rows_allow_256bit(const void* x, const void* xt, const void* g, int64_t pitch, int32_t dtype) {
    return rows_32B_aligned(x, xt, g, pitch, dtype);
}

int launch_events(const EventLaunch& L, const DeviceInfo& dev, void* stream_) {
    if (L.n_items <= 0) return 0;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (L.variant == A2_NO_MOMENTUM) {
        const bool wide_x = rows_32B_aligned(L.x, nullptr, L.g, L.pitch, L.dtype);
        if (L.dtype == A2_BF16) {
            static const bool force_narrow = a2::tuning_env("A2CID2_FORCE_128BIT") != nullptr;  // tuning override
            const uintptr_t bits = reinterpret_cast<uintptr_t>(L.x) | reinterpret_cast<uintptr_t>(L.g);
            const bool wide_bf16 = !force_narrow && bits % 32 == 0 && (L.pitch * 2) % 32 == 0;
            if (L.max_workers >= 3)
                return wide_bf16 ? launch_plain_bf16<8, 3>(L, dev, stream) : launch_plain_bf16<4, 3>(L, dev, stream);
            return wide_bf16 ? launch_plain_bf16<8, 2>(L, dev, stream) : launch_plain_bf16<4, 2>(L, dev, stream);
        }
        if (L.max_workers >= 3)
            return wide_x ? launch_plain_t<float, 32, 3>(L, dev, stream) : launch_plain_t<float, 16, 3>(L, dev, stream);
        return wide_x ? launch_plain_t<float, 32, 2>(L, dev, stream) : launch_plain_t<float, 16, 2>(L, dev, stream);
    }
    const bool wide = rows_32B_aligned(L.x, L.xt, L.g, L.pitch, L.dtype);
    if (L.round_per_store) {  // one kernel serves every item width in this mode; the caller has checked the rest
        if (!wide || L.dtype == A2_BF16) return (int)cudaErrorInvalidValue;
        return launch_events_pairs4(L, dev, stream);
    }
    if (L.max_workers >= 4 && L.dtype != A2_BF16) {
        static const bool narrow4 = a2::tuning_env("A2CID2_EVENT4_128BIT") != nullptr;  // tuning override
        if (wide && !narrow4) return launch_events_pairs4(L, dev, stream);
        return launch_events_t<float, 16, 4, kEventThreads, A2_EVENT4_UNROLL_128>(L, dev, stream);
    }
    if (L.max_workers >= 3) {
        if (L.dtype == A2_BF16) {
            static const bool force_narrow = a2::tuning_env("A2CID2_FORCE_128BIT") != nullptr;  // tuning override
            const uintptr_t bits = reinterpret_cast<uintptr_t>(L.x) | reinterpret_cast<uintptr_t>(L.xt) |
                                   reinterpret_cast<uintptr_t>(L.g);
            const bool wide_bf16 = !force_narrow && bits % 32 == 0 && (L.pitch * 2) % 32 == 0;
            return wide_bf16 ? launch_bf16_packed<8>(L, dev, stream) : launch_bf16_packed<4>(L, dev, stream);
        }
        return wide ? launch_events_t<float, 32, 3>(L, dev, stream) : launch_events_t<float, 16, 3>(L, dev, stream);
    }
    if (L.dtype == A2_BF16) return launch_events_t<__nv_bfloat16, 16, 2>(L, dev, stream);
    return wide ? launch_events_t<float, 32, 2>(L, dev, stream) : launch_events_t<float, 16, 2>(L, dev, stream);
}

int consensus_grid(const DeviceInfo& dev) { return dev.sm_count * dev.consensus_ctas_per_sm; }

int launch_consensus(const void* x, const void* xt, int64_t pitch, int32_t n, int64_t d, int32_t dtype, double eta,
                     const double* dt, double* partials, int n_partials, double* out, void* stream_) {
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const bool wide = rows_32B_aligned(x, xt, nullptr, pitch, dtype);
    const int sms = n_partials / 8 > 0 ? n_partials / 8 : 1;  // the scratch holds 8 partial sums per SM
    int used;
    if (dtype == A2_BF16) {
        used = launch_consensus_partial_t<__nv_bfloat16, 16>(x, xt, pitch, n, d, eta, dt, partials, n_partials, sms, stream);
    } else {
        if (wide) used = launch_consensus_partial_t<float, 32>(x, xt, pitch, n, d, eta, dt, partials, n_partials, sms, stream);
        else used = launch_consensus_partial_t<float, 16>(x, xt, pitch, n, d, eta, dt, partials, n_partials, sms, stream);
    }
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return (int)e;
    k_consensus_final<<<1, kThreads, 0, stream>>>(partials, used, out);
    return (int)cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// Resident mode: one launch for a whole event stream.
//
// Every operation of the method is element-wise over the parameter dimension, so a column never
// needs another column. A thread therefore owns one column of a 256-column tile for ALL n workers:
// it loads x[:, c] and x~[:, c] into its own lane of shared memory (used as a register file that
// can be indexed by worker), walks the events in stream order, and writes the column back. No thread
// reads what another thread wrote: there is no barrier, no flag and no wait anywhere. The gradient
// rows an event needs come from a small cache in shared memory that is refilled chunk by chunk of the
// stream (the host cut the stream so that a chunk's distinct rows fit). The state crosses HBM once per
// call, gradient rows once per use; the rest is shared-memory traffic and ALU work.
// ---------------------------------------------------------------------------------------------
namespace {

__global__ void __launch_bounds__(kThreads) k_resident_prepare(const DevItem* __restrict__ items,
                                                             const DevOp* __restrict__ ops, int n_events, double eta,
                                                             ResEv* __restrict__ out) {
    const int e = blockIdx.x * kThreads + threadIdx.x;
    if (e >= n_events) return;
    const DevItem it = items[e];
    const DevOp op = ops[e];
    ResEv r;
    r.a = (int16_t)it.a;
    r.b = (int16_t)it.b;
    r.g = (int16_t)it.slot_b;  // cache index of the gradient row (set by the host for gradient events)
    r.kind = (int16_t)op.kind;
    r.ca = (float)mix_coeff(eta, op.t - op.t_prev_a);
    r.cb = op.kind == A2_OP_COMM ? (float)mix_coeff(eta, op.t - op.t_prev_b) : 0.f;
    out[e] = r;
}

template <typename T> __device__ __forceinline__ float widen1(T v);
template <> __device__ __forceinline__ float widen1<float>(float v) { return v; }
template <> __device__ __forceinline__ float widen1<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T narrow1(float v);
template <> __device__ __forceinline__ float narrow1<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 narrow1<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

struct ResidentArgs {
    void* x;
    void* xt;
    const void* g;
    long long pitch;
    long long n_tiles;
    int n;
    const ResEv* events;
    const ResChunk* chunks;
    const int* g_rows;
    int n_chunks;
    float alpha, alpha_tilde, gamma;
    int msg_before_mix;
};

template <typename T>
__global__ void __launch_bounds__(kResidentCols) k_resident(const ResidentArgs p) {
    extern __shared__ float s_tile[];  // [n][256] x, [n][256] x~, [cache][256] gradient rows
    float* const sX = s_tile + threadIdx.x;
    float* const sXt = sX + (size_t)p.n * kResidentCols;
    float* const sG = sXt + (size_t)p.n * kResidentCols;
    T* const X = static_cast<T*>(p.x);
    T* const Xt = static_cast<T*>(p.xt);
    const T* const G = static_cast<const T*>(p.g);
    const int lane = threadIdx.x & 31;
    const float ngamma = -p.gamma;
    const bool before = p.msg_before_mix != 0;

    for (long long tile = blockIdx.x; tile < p.n_tiles; tile += gridDim.x) {
        const long long col = tile * kResidentCols + threadIdx.x;
        const bool active = col < p.pitch;  // padding columns are carried along; nothing past the pitch is touched
#pragma unroll 8
        for (int i = 0; i < p.n; ++i) {
            sX[i * kResidentCols] = active ? widen1<T>(__ldcs(X + (long long)i * p.pitch + col)) : 0.f;
            sXt[i * kResidentCols] = active ? widen1<T>(__ldcs(Xt + (long long)i * p.pitch + col)) : 0.f;
        }
        for (int c = 0; c < p.n_chunks; ++c) {
            const ResChunk ch = p.chunks[c];
#pragma unroll 4
            for (int k = 0; k < ch.g_count; ++k)
                sG[k * kResidentCols] = active ? widen1<T>(__ldg(G + (long long)p.g_rows[ch.g_begin + k] * p.pitch + col)) : 0.f;
            for (int e0 = ch.ev_begin; e0 < ch.ev_end; e0 += 32) {
                // a warp fetches 32 descriptors with one coalesced load and hands them round by shuffle
                int4 mine = make_int4(0, 0, 0, 0);
                if (e0 + lane < ch.ev_end) mine = __ldg(reinterpret_cast<const int4*>(p.events) + e0 + lane);
                const int cnt = min(32, ch.ev_end - e0);
                for (int l = 0; l < cnt; ++l) {
                    const int w0 = __shfl_sync(0xffffffffu, mine.x, l);
                    const int w1 = __shfl_sync(0xffffffffu, mine.y, l);
                    const float ca = __int_as_float(__shfl_sync(0xffffffffu, mine.z, l));
                    const float cb = __int_as_float(__shfl_sync(0xffffffffu, mine.w, l));
                    const int a = (int)(short)(w0 & 0xFFFF), b = (int)(short)(w0 >> 16);
                    const int gi = (int)(short)(w1 & 0xFFFF), kind = (int)(short)(w1 >> 16);
                    float xa = sX[a * kResidentCols], xta = sXt[a * kResidentCols];
                    if (kind == A2_OP_COMM) {
                        float xb = sX[b * kResidentCols], xtb = sXt[b * kResidentCols];
                        comm_elem<sizeof(T) == 4>(xa, xta, xb, xtb, ca, cb, p.alpha, p.alpha_tilde, before);
                        sX[b * kResidentCols] = xb;
                        sXt[b * kResidentCols] = xtb;
                    } else {
                        grad_elem<sizeof(T) == 4>(xa, xta, ca, ngamma, sG[gi * kResidentCols]);
                    }
                    sX[a * kResidentCols] = xa;
                    sXt[a * kResidentCols] = xta;
                }
            }
        }
        if (active) {
#pragma unroll 8
            for (int i = 0; i < p.n; ++i) {
                __stcs(X + (long long)i * p.pitch + col, narrow1<T>(sX[i * kResidentCols]));
                __stcs(Xt + (long long)i * p.pitch + col, narrow1<T>(sXt[i * kResidentCols]));
            }
        }
    }
}

template <typename T>
int launch_resident_t(const ResidentLaunch& L, const DeviceInfo& dev, cudaStream_t stream) {
    const size_t smem = (size_t)(2 * L.n + L.cache_rows) * kResidentCols * sizeof(float);
    cudaError_t e = cudaFuncSetAttribute(k_resident<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return (int)e;
    int occ = 0;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, k_resident<T>, kResidentCols, smem);
    if (e != cudaSuccess) return (int)e;
    if (occ < 1) return (int)cudaErrorInvalidConfiguration;
    ResidentArgs a;
    a.x = L.x; a.xt = L.xt; a.g = L.g; a.pitch = L.pitch;
    a.n_tiles = (L.d + kResidentCols - 1) / kResidentCols;
    a.n = L.n; a.events = L.events; a.chunks = L.chunks; a.g_rows = L.g_rows; a.n_chunks = L.n_chunks;
    a.alpha = L.alpha; a.alpha_tilde = L.alpha_tilde; a.gamma = L.gamma;
    a.msg_before_mix = L.variant == A2_MSG_BEFORE_MIX;
    long long grid = (long long)dev.sm_count * occ;
    if (grid > a.n_tiles) grid = a.n_tiles;
    k_resident<T><<<(unsigned)grid, kResidentCols, smem, stream>>>(a);
    return (int)cudaGetLastError();
}

}  // namespace

int resident_cache_rows(int32_t n, int32_t n_grad_slots) {
    const int room = kResidentMaxRows - 2 * n;
    if (room < kResidentMinCache) return 0;
    int want = n_grad_slots < kResidentMinCache ? kResidentMinCache : n_grad_slots;
    // more cache rows than needed only lowers occupancy; 64 rows are refilled every few hundred events at most
    if (want > 64) want = 64;
    return want < room ? want : room;
}

int launch_resident(const ResidentLaunch& L, const DeviceInfo& dev, void* stream_) {
    if (L.n_events <= 0) return 0;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const int blocks = (L.n_events + kThreads - 1) / kThreads;
    k_resident_prepare<<<blocks, kThreads, 0, stream>>>(L.items, L.ops, L.n_events, L.eta, L.events);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return (int)e;
    if (L.dtype == A2_BF16) return launch_resident_t<__nv_bfloat16>(L, dev, stream);
    return launch_resident_t<float>(L, dev, stream);
}

// ---------------------------------------------------------------------------------------------
// Consensus distance without any allocation: the per-block partial sums live in a fixed array
// that is part of the loaded library image instead of in memory obtained at run time.
// ---------------------------------------------------------------------------------------------
namespace {

constexpr int kStaticVecPerBlock = 4096;  // 128-bit vectors of one row handled by one block
static __device__ __align__(256) double g_static_partials[kStaticMaxPartials];

// Host code may not hand `g_static_partials` to a kernel: in host code that name is only a
// stand-in for the device symbol. Its device address is looked up once per device, with that
// device current, and cached here.
constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;
double* g_static_addr[kMaxDevices] = {};

}  // namespace

int launch_consensus_static(const void* x, int64_t pitch, int32_t n, int64_t d, int32_t dtype, double* out_device,
                            void* stream_, int* n_partials_out) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return (int)e;
    if (dev < 0 || dev >= kMaxDevices) return (int)cudaErrorInvalidDevice;
    double* partials = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_static_mutex);
        if (!g_static_addr[dev]) {
            void* p = nullptr;
            e = cudaGetSymbolAddress(&p, g_static_partials);
            if (e != cudaSuccess) return (int)e;
            // With lazy module loading a kernel's code reaches the device when it is first needed. Asking for the
            // attributes of the three kernels this entry point can launch (both storage types) loads them now, so
            // that a later call with the other storage type brings nothing new onto the device either.
            cudaFuncAttributes fa;
            if ((e = cudaFuncGetAttributes(&fa, k_consensus_partial<float, 16, false>)) != cudaSuccess) return (int)e;
            if ((e = cudaFuncGetAttributes(&fa, k_consensus_partial<__nv_bfloat16, 16, false>)) != cudaSuccess) return (int)e;
            if ((e = cudaFuncGetAttributes(&fa, k_consensus_final)) != cudaSuccess) return (int)e;
            g_static_addr[dev] = static_cast<double*>(p);
        }
        partials = g_static_addr[dev];
    }
    const int vec = dtype == A2_BF16 ? 8 : 4;
    const int64_t n_vec = (d + vec - 1) / vec;
    const int64_t blocks = (n_vec + kStaticVecPerBlock - 1) / kStaticVecPerBlock;
    if (blocks < 1 || blocks > kStaticMaxPartials) return (int)cudaErrorInvalidValue;  // checked by the caller too
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    // every block overwrites its own partial and the final pass reads exactly `blocks` of them,
    // so nothing left in the array by an earlier call is ever read
    if (dtype == A2_BF16)
        k_consensus_partial<__nv_bfloat16, 16, false><<<(unsigned)blocks, kThreads, 0, stream>>>(
            static_cast<const __nv_bfloat16*>(x), nullptr, pitch, n, d, 0.0, nullptr, partials);
    else
        k_consensus_partial<float, 16, false><<<(unsigned)blocks, kThreads, 0, stream>>>(
            static_cast<const float*>(x), nullptr, pitch, n, d, 0.0, nullptr, partials);
    e = cudaGetLastError();
    if (e != cudaSuccess) return (int)e;
    k_consensus_final<<<1, kThreads, 0, stream>>>(partials, (int)blocks, out_device);
    if (n_partials_out) *n_partials_out = (int)blocks;
    return (int)cudaGetLastError();
}

int64_t consensus_static_max_columns(int32_t dtype) {
    return (int64_t)kStaticMaxPartials * kStaticVecPerBlock * (dtype == A2_BF16 ? 8 : 4);
}

}  // namespace a2
