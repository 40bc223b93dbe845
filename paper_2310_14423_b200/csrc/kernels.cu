// CUDA kernels of the Local-OPT hot path for sm_100a: the fused local step (Eq. 1 of arXiv 2310.14423, with the
// synthetic gradient generated in registers) and the replica-axis mean that ends a round (Algorithm 2).
//
// Both are pure HBM streams over [K, P] fp32 slabs: nothing here is a contraction, so there are no tensor-core
// instructions.  A thread owns one 16-byte column (4 consecutive coordinates) for ALL K rows: lambda / theta_star
// are fetched once per column instead of once per worker, every global access is a 128-bit LDG/STG on a
// 16-byte boundary, a warp touches 512 contiguous bytes per row, and the step kernel keeps the loads of eight rows
// per thread in flight through a cp.async ring in shared memory to cover HBM latency.
#include <cuda_runtime.h>

#include <atomic>
#include <cstdint>
#include <cstring>

#include "internal.h"

namespace qsr {
namespace {

// ---------------------------------------------------------------------------------------------- noise

// Philox-4x32 with 10 rounds (Salmon et al., SC'11): 128-bit counter, 64-bit key.  The key schedule
// (key + r * Weyl constant) does not depend on the counter, so the host evaluates it once per launch and the ten
// round keys arrive as kernel arguments: a round is two 32x32->64 multiplies and two three-input XORs.
__device__ __forceinline__ uint4 philox4x32_10(uint4 c, const uint32_t (&rk)[20])
{
    constexpr uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint64_t p0 = uint64_t(M0) * c.x, p1 = uint64_t(M1) * c.z;
        c = make_uint4(uint32_t(p1 >> 32) ^ c.y ^ rk[2 * r], uint32_t(p1), uint32_t(p0 >> 32) ^ c.w ^ rk[2 * r + 1],
                       uint32_t(p0));
    }
    return c;
}

// Square root and reciprocal as ONE special-function instruction each.  The IEEE forms are sequences of about 8 and
// 10 instructions with a slow-path branch, and even the .approx forms carry extra scaling code for subnormal
// operands unless they are the flush-to-zero variants used here.  Flushing is harmless at both call sites: the
// Box-Muller radicand lies in [1e-7, 34], and a second moment below 1e-38 has a square root far below eps either way.
// Measured on B200 over 2^24 inputs: relative error of sqrt.approx at most 1.0e-7 (mean -1.2e-8), of the reciprocal
// at most 1.5e-7 (mean 3e-12) -- rounding-level, far inside the parity bound.
__device__ __forceinline__ float sqrt_fast(float x)
{
    float y;
    asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float rcp_fast(float x)
{
    float y;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// -2 ln(u) for u = (a + 1/2) / 2^23, a = the top 23 bits of w: u is exact in fp32 and lies in [2^-24, 1 - 2^-24].
// The 23 bits are dropped into the mantissa of a float in [1, 2) and shifted down by an exact subtraction (no
// integer-to-float conversion).  ln(u) = e ln 2 + ln(m) with u = m 2^e, m in [2/3, 4/3); ln(m) = f + f^2 Q(f), f = m - 1,
// Q a degree-7 minimax fit of (ln(1+f) - f) / f^2 on [-1/3, 1/3] (|error| < 1.7e-7, i.e. < 6e-8 relative to ln m).
// The input range is known, so none of a general logf's tests for zero, negative, infinite or subnormal arguments is
// needed.  Over all 2^23 values of a the relative error of the result is below 1.0e-7 with no bias in the mean.
__device__ __forceinline__ float neg2_log_unit(uint32_t w)
{
    const float u = __uint_as_float(0x3f800000u | (w >> 9)) - (1.0f - 0x1p-24f);      // (a + 1/2) / 2^23, exact
    const int t = __float_as_int(u) - 0x3f2aaaab;                                     // 0x3f2aaaab: bits of 2/3
    const float m = __int_as_float((t & 0x007fffff) + 0x3f2aaaab);
    const float e = __int_as_float(0x4b400000 + (t >> 23)) - 12582912.0f;             // exponent as a float, exact
    const float f = m - 1.0f;
    float q = 0.14067277312278748f;
    q = fmaf(q, f, -0.15009641647338867f);
    q = fmaf(q, f, 0.13995099067687988f);
    q = fmaf(q, f, -0.16489295661449432f);
    q = fmaf(q, f, 0.20010477304458618f);
    q = fmaf(q, f, -0.2500377893447876f);
    q = fmaf(q, f, 0.3333323299884796f);
    q = fmaf(q, f, -0.49999991059303284f);
    const float ln_m = fmaf(f * f, q, f);
    return -2.0f * fmaf(e, 0.6931471805599453f, ln_m);
}

// cos and sin of the angle 2 pi (b + 1/2) / 2^23, b = the top 23 bits of w.  In quarter turns the angle is
// x = (b + 1/2) / 2^21 = n + y with n = round(x) and y in (-1/2, 1/2); n mod 4 is the top two bits of
// w + 2^29 (the addition wraps at a full turn), the next 21 bits are y + 1/2 up to the half-unit offset, and they
// become a float by the same mantissa trick, so the argument reduction is exact and costs four integer/float
// instructions.  sin(pi/2 y) and cos(pi/2 y) are degree-7 / degree-8 minimax polynomials (|error| < 3e-9 / 2e-10);
// the quadrant swaps them and sets the signs with the same top bits.  Over all 2^23 angles: |error| < 9e-8, mean 0.
__device__ __forceinline__ void sincos_turn_bits(uint32_t w, float &sin_out, float &cos_out)
{
    const uint32_t t = w + 0x20000000u;
    const float y = __uint_as_float(((t >> 7) & 0x007ffffcu) | 0x3f800000u) - (1.5f - 0x1p-22f);
    const float y2 = y * y;
    float ps = -0.004602177068591118f;
    ps = fmaf(ps, y2, 0.07968022674322128f);
    ps = fmaf(ps, y2, -0.6459634900093079f);
    ps = fmaf(ps, y2, 1.5707963705062866f);
    const float s = y * ps;
    float pc = 0.0009067608625628054f;
    pc = fmaf(pc, y2, -0.020861538127064705f);
    pc = fmaf(pc, y2, 0.253669410943985f);
    pc = fmaf(pc, y2, -1.2337005138397217f);
    const float c = fmaf(pc, y2, 1.0f);
    const bool odd = (t & 0x40000000u) != 0;                  // n odd: sine and cosine trade places
    const float c0 = odd ? s : c, s0 = odd ? c : s;
    // signs: sin < 0 for n in {2, 3} (bit 31 of t), cos < 0 for n in {1, 2} (bit 31 of t + 2^30)
    sin_out = __uint_as_float(__float_as_uint(s0) ^ (t & 0x80000000u));
    cos_out = __uint_as_float(__float_as_uint(c0) ^ ((t + 0x40000000u) & 0x80000000u));
}

// Box-Muller on two words: uniforms are (top 23 bits + 1/2) / 2^23, exact in fp32 and never 0 or 1.
// Both transcendental parts are written for exactly these inputs (see above) rather than taken from the math library:
// the generic logf and sincospif cost about twice the instructions, and the step kernel is bound by instruction issue
// almost as much as by memory.  Their errors stay rounding-sized and unbiased; a bias of 1e-8 in the noise would move
// the fixed point of a coordinate with curvature 1e-3 by 1e-5 * sigma, which is why the hardware's approximate
// sine/cosine (biased by about -1.3e-8 on this grid) is not used.
__device__ __forceinline__ void box_muller(uint32_t wa, uint32_t wb, float &z_cos, float &z_sin)
{
    const float radius = sqrt_fast(neg2_log_unit(wa));
    float s, c;
    sincos_turn_bits(wb, s, c);
    z_cos = radius * c;
    z_sin = radius * s;
}

// Four standard normals for coordinates 4j .. 4j+3 of one worker at one step.
__device__ __forceinline__ float4 noise4(int64_t j, uint32_t step, uint32_t worker, const uint32_t (&rk)[20])
{
    const uint4 r = philox4x32_10(make_uint4(uint32_t(j), uint32_t(uint64_t(j) >> 32), step, worker), rk);
    float4 z;
    box_muller(r.x, r.y, z.x, z.y);
    box_muller(r.z, r.w, z.z, z.w);
    return z;
}

// ---------------------------------------------------------------------------------------------- OPT (Eq. 1)

// `wdv` is the weight-decay scalar of this coordinate's tensor: wd for SGD, eta*wd for AdamW, each times the
// tensor's scale (1 when no tensor table is set).
template <int OPT>
__device__ __forceinline__ void opt_update(float &theta, float &a, float &b, float g, const StepParams &p, float wdv)
{
    if (OPT == QSR_OPT_SGDM) {
        g = fmaf(wdv, theta, g);           // L2 weight decay enters the gradient
        a = fmaf(p.mu, a, g);              // heavy-ball buffer
        theta = fmaf(-p.eta, a, theta);
    } else {
        // Moments in the interpolation form x <- x + (1 - beta)(y - x): a constant gradient is then a fixed point
        // exactly (m = g, v = g^2), whereas beta*x + (1 - beta)*y with both factors rounded to fp32 has fixed point
        // y * fl(1 - beta) / (1 - fl(beta)), off by 2e-7 for beta1 = 0.9 and 1.3e-5 for beta2 = 0.999.
        a = fmaf(p.omb1, g - a, a);
        b = fmaf(p.omb2, fmaf(g, g, -b), b);
        const float denom = fmaf(sqrt_fast(b), p.inv_sqrt_bc2, p.eps);
        // theta*(1 - eta*wd) - step_size*m/denom as ONE subtraction from theta.  Forming 1 - eta*wd in fp32 would
        // keep only ~2^-24 of absolute precision on a term of size eta*wd, and the product theta*(1 - eta*wd) has
        // near-ties that round the same way step after step when theta sits just above a power of two; both show up
        // as a drift of a few 1e-5 over thousands of small steps.  The decay and the update are summed first instead.
        theta -= fmaf(wdv, theta, (p.step_size * a) * rcp_fast(denom));
    }
}

// Weight-decay scalar for the column that starts at coordinate i0: binary search of the tensor that holds it
// (tensor_end is ascending, every entry but the last a multiple of 4, so a column never straddles two tensors).
template <int OPT>
__device__ __forceinline__ float weight_decay_at(const StepParams &p, int64_t i0)
{
    const float base = OPT == QSR_OPT_SGDM ? p.wd : p.eta_wd;
    if (p.n_tensors == 0) return base;
    int lo = 0, hi = p.n_tensors - 1;
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (__ldg(p.tensor_end + mid) > i0) hi = mid;
        else lo = mid + 1;
    }
    return base * __ldg(p.wd_scale + lo);
}

__device__ __forceinline__ float4 ld4(const float *p) { return *reinterpret_cast<const float4 *>(p); }
__device__ __forceinline__ void st4(float *p, float4 v) { *reinterpret_cast<float4 *>(p) = v; }

__device__ __forceinline__ float4 add4(float4 x, float4 y) { return make_float4(x.x + y.x, x.y + y.y, x.z + y.z, x.w + y.w); }
__device__ __forceinline__ float4 div4(float4 x, float d) { return make_float4(x.x / d, x.y / d, x.z / d, x.w / d); }

// Asynchronous 16-byte copies global -> shared (LDGSTS): the data does not pass through registers, so a thread can
// keep many rows in flight at no register cost.  Each thread only ever reads back the slots it filled itself, so
// cp.async.wait_group (which orders a thread's own copies) is all the synchronization there is: no barriers, no waits
// on other threads, nothing that could spin.
__device__ __forceinline__ void cp_async16(float4 *smem_dst, const float *gmem_src)
{
    const unsigned dst = static_cast<unsigned>(__cvta_generic_to_shared(smem_dst));
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait_all_but() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// ---------------------------------------------------------------------------------------------- packed arithmetic
//
// The kernels that are bound by instruction issue rather than by memory -- Algorithm 1's step, the
// gradient-norm pass of clipping and the register-resident launches -- evaluate the noise, the gradient and the
// optimizer update two lanes at a time.  Every component is rounded exactly like its scalar form, so the results are
// the bits of noise4 / opt_update (the tests that compare these kernels with the per-step kernel bit for bit cover it).
// The memory-bound step kernel keeps the scalar forms: packing does not change its time, and its round-end instance
// loses half a percent to the register pairs.  Measured on B200: Algorithm-1 step 1.827 -> 1.701 ms at the ViT-B/16
// shape and 1.260 -> 1.130 ms at the ResNet-152 shape, clipped step 8.00 -> 7.77 ms, resident launches 14.6 -> 13.6 us
// per step at K = 8, P = 2^20.
//
// sm_100 executes two independent fp32 operations per lane in one instruction (fma / add / mul on a register pair),
// each component rounded exactly like its scalar form; what comes in pairs here are the two Box-Muller transforms of
// a Philox block and the four coordinates of a column.
__device__ __forceinline__ float2 fma2(float2 a, float2 b, float2 c) { return __ffma2_rn(a, b, c); }
__device__ __forceinline__ float2 mul2(float2 a, float2 b) { return __fmul2_rn(a, b); }
__device__ __forceinline__ float2 add2(float2 a, float2 b) { return __fadd2_rn(a, b); }
__device__ __forceinline__ float2 sub2(float2 a, float2 b) { return __fadd2_rn(a, make_float2(-b.x, -b.y)); }
__device__ __forceinline__ float2 both(float x) { return make_float2(x, x); }

// neg2_log_unit for two words at once (same operations per component).
__device__ __forceinline__ float2 neg2_log_unit2(uint32_t w0, uint32_t w1)
{
    const float2 u = add2(make_float2(__uint_as_float(0x3f800000u | (w0 >> 9)), __uint_as_float(0x3f800000u | (w1 >> 9))),
                          both(-(1.0f - 0x1p-24f)));
    const int t0 = __float_as_int(u.x) - 0x3f2aaaab, t1 = __float_as_int(u.y) - 0x3f2aaaab;
    const float2 m = make_float2(__int_as_float((t0 & 0x007fffff) + 0x3f2aaaab), __int_as_float((t1 & 0x007fffff) + 0x3f2aaaab));
    // The two arithmetic shifts are written in PTX: written as `t >> 23` next to each other, nvcc 12.9 drops the
    // shift of the first one (the pair comes out as (t0, t1 >> 23); seen on sm_100a at -O3, scalar code unaffected).
    int e0, e1;
    asm("shr.s32 %0, %1, 23;" : "=r"(e0) : "r"(t0));
    asm("shr.s32 %0, %1, 23;" : "=r"(e1) : "r"(t1));
    const float2 e = add2(make_float2(__int_as_float(0x4b400000 + e0), __int_as_float(0x4b400000 + e1)), both(-12582912.0f));
    const float2 f = add2(m, both(-1.0f));
    float2 q = both(0.14067277312278748f);
    q = fma2(q, f, both(-0.15009641647338867f));
    q = fma2(q, f, both(0.13995099067687988f));
    q = fma2(q, f, both(-0.16489295661449432f));
    q = fma2(q, f, both(0.20010477304458618f));
    q = fma2(q, f, both(-0.2500377893447876f));
    q = fma2(q, f, both(0.3333323299884796f));
    q = fma2(q, f, both(-0.49999991059303284f));
    const float2 ln_m = fma2(mul2(f, f), q, f);
    return mul2(both(-2.0f), fma2(e, both(0.6931471805599453f), ln_m));
}

// sincos_turn_bits for two words at once.
__device__ __forceinline__ void sincos_turn_bits2(uint32_t w0, uint32_t w1, float2 &sin_out, float2 &cos_out)
{
    const uint32_t t0 = w0 + 0x20000000u, t1 = w1 + 0x20000000u;
    const float2 y = add2(make_float2(__uint_as_float(((t0 >> 7) & 0x007ffffcu) | 0x3f800000u),
                                      __uint_as_float(((t1 >> 7) & 0x007ffffcu) | 0x3f800000u)),
                          both(-(1.5f - 0x1p-22f)));
    const float2 y2 = mul2(y, y);
    float2 ps = both(-0.004602177068591118f);
    ps = fma2(ps, y2, both(0.07968022674322128f));
    ps = fma2(ps, y2, both(-0.6459634900093079f));
    ps = fma2(ps, y2, both(1.5707963705062866f));
    const float2 s = mul2(y, ps);
    float2 pc = both(0.0009067608625628054f);
    pc = fma2(pc, y2, both(-0.020861538127064705f));
    pc = fma2(pc, y2, both(0.253669410943985f));
    pc = fma2(pc, y2, both(-1.2337005138397217f));
    const float2 c = fma2(pc, y2, both(1.0f));
    const bool odd0 = (t0 & 0x40000000u) != 0, odd1 = (t1 & 0x40000000u) != 0;
    const float c0 = odd0 ? s.x : c.x, s0 = odd0 ? c.x : s.x;
    const float c1 = odd1 ? s.y : c.y, s1 = odd1 ? c.y : s.y;
    sin_out = make_float2(__uint_as_float(__float_as_uint(s0) ^ (t0 & 0x80000000u)),
                          __uint_as_float(__float_as_uint(s1) ^ (t1 & 0x80000000u)));
    cos_out = make_float2(__uint_as_float(__float_as_uint(c0) ^ ((t0 + 0x40000000u) & 0x80000000u)),
                          __uint_as_float(__float_as_uint(c1) ^ ((t1 + 0x40000000u) & 0x80000000u)));
}

// noise4 with the block's two Box-Muller transforms (words 0,1 and words 2,3) side by side in the two lanes of the
// packed operations: the same bits as noise4.
__device__ __forceinline__ float4 noise4_packed(int64_t j, uint32_t step, uint32_t worker, const uint32_t (&rk)[20])
{
    const uint4 r = philox4x32_10(make_uint4(uint32_t(j), uint32_t(uint64_t(j) >> 32), step, worker), rk);
    const float2 n2l = neg2_log_unit2(r.x, r.z);
    const float2 radius = make_float2(sqrt_fast(n2l.x), sqrt_fast(n2l.y));
    float2 s, c;
    sincos_turn_bits2(r.y, r.w, s, c);
    const float2 zc = mul2(radius, c), zs = mul2(radius, s);
    return make_float4(zc.x, zs.x, zc.y, zs.y);
}

// The synthetic gradient of four coordinates: lambda (theta - theta_star) + sigma z.
__device__ __forceinline__ float4 gradient4(float sigma, float4 z, float4 lam, float4 th, float4 ths)
{
    const float2 lo = fma2(both(sigma), make_float2(z.x, z.y),
                           mul2(make_float2(lam.x, lam.y), sub2(make_float2(th.x, th.y), make_float2(ths.x, ths.y))));
    const float2 hi = fma2(both(sigma), make_float2(z.z, z.w),
                           mul2(make_float2(lam.z, lam.w), sub2(make_float2(th.z, th.w), make_float2(ths.z, ths.w))));
    return make_float4(lo.x, lo.y, hi.x, hi.y);
}

// opt_update on two coordinates at once (same operations per component as the scalar form above).
template <int OPT>
__device__ __forceinline__ void opt_update2(float2 &theta, float2 &a, float2 &b, float2 g, const StepParams &p, float wdv)
{
    if (OPT == QSR_OPT_SGDM) {
        g = fma2(both(wdv), theta, g);
        a = fma2(both(p.mu), a, g);
        theta = fma2(both(-p.eta), a, theta);
    } else {
        a = fma2(both(p.omb1), sub2(g, a), a);
        b = fma2(both(p.omb2), fma2(g, g, make_float2(-b.x, -b.y)), b);
        const float2 denom = fma2(make_float2(sqrt_fast(b.x), sqrt_fast(b.y)), both(p.inv_sqrt_bc2), both(p.eps));
        const float2 step = mul2(mul2(both(p.step_size), a), make_float2(rcp_fast(denom.x), rcp_fast(denom.y)));
        theta = sub2(theta, fma2(both(wdv), theta, step));
    }
}

template <int OPT>
__device__ __forceinline__ void opt_update4(float4 &th, float4 &a, float4 &b, float4 g, const StepParams &p, float wdv)
{
    float2 t0 = make_float2(th.x, th.y), t1 = make_float2(th.z, th.w);
    float2 a0 = make_float2(a.x, a.y), a1 = make_float2(a.z, a.w);
    float2 b0 = make_float2(b.x, b.y), b1 = make_float2(b.z, b.w);
    opt_update2<OPT>(t0, a0, b0, make_float2(g.x, g.y), p, wdv);
    opt_update2<OPT>(t1, a1, b1, make_float2(g.z, g.w), p, wdv);
    th = make_float4(t0.x, t0.y, t1.x, t1.y);
    a = make_float4(a0.x, a0.y, a1.x, a1.y);
    b = make_float4(b0.x, b0.y, b1.x, b1.y);
}

// 16-byte load when the whole column lies inside the row, scalar loads (zeros beyond P) for the ragged last column.
__device__ __forceinline__ float4 ld4_guarded(const float *q, int valid)
{
    if (valid == 4) return ld4(q);
    return make_float4(q[0], valid > 1 ? q[1] : 0.f, valid > 2 ? q[2] : 0.f, 0.f);
}

// Sum of squares of worker k's generated gradient over the (up to four) coordinates of column j at step `step`, the
// parameters given in th: what the global norm of gradient clipping (App. C.2) is made of.  One definition for the
// norm pass and for the step kernel that computes the next step's norms on the side, so that both give the same bits.
__device__ __forceinline__ float column_sq(const StepParams &p, int64_t j, uint32_t step, int k, float4 th, float4 lam,
                                           float4 ths, int valid)
{
    const float4 z = noise4_packed(j, step, p.worker0 + uint32_t(k), p.round_key);
    float4 g = gradient4(p.sigma, z, lam, th, ths);
    if (valid < 4) {                   // ragged last column: the lanes beyond P do not count
        g.y = valid > 1 ? g.y : 0.f;
        g.z = valid > 2 ? g.z : 0.f;
        g.w = 0.f;
    }
    return fmaf(g.x, g.x, g.y * g.y) + fmaf(g.z, g.z, g.w * g.w);
}

// Block reduction of per-thread values acc[row][thread] to partial[block][row]: warp w folds rows w, w + n_warps, ...
// in a fixed order (lanes stride over the threads, then a butterfly), so the result does not depend on timing.
__device__ __forceinline__ void reduce_rows_to_partials(const float *acc, int rows, float *partial)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
    for (int r = warp; r < rows; r += n_warps) {
        float v = 0.f;
        for (int t = lane; t < int(blockDim.x); t += 32) v += acc[r * blockDim.x + t];
        for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        if (lane == 0) partial[int64_t(blockIdx.x) * rows + r] = v;
    }
}

// One local step of all K workers.
//
// Memory pipeline.  A thread owns one 16-byte column and walks down the K rows.  Row k's operands (theta, state1,
// [state2], [gradient]) are fetched by cp.async into the thread's private slots of a STAGES-deep ring in shared
// memory; the ring is filled STAGES rows ahead, and as soon as a row has been copied to registers its slot is
// refilled with row k + STAGES.  With 256 threads, 8 stages and AdamW's three operands a CTA holds 96 KB of loads in
// flight (two CTAs per SM), against about 60 KB per SM when the rows in flight had to live in registers; on B200
// that took the sustained ViT-B/16-shaped AdamW step from 5.6 ms to 5.35 ms, and trimming the instruction stream
// (see the noise section) brought it to 5.3 ms, 97-98 % of the rate of a device-to-device copy.
// Results go straight from registers to global memory with 128-bit stores.
//
// Round end.  With FUSE != 0 the step is the last of its round and the kernel also ends the round (Algorithm 2's
// averaging, state kept per worker): the thread that owns a column sees every worker's new parameters anyway, so it
// sums them as it goes (k ascending, fp32: the order of the stand-alone sync kernel, hence the same bits).
// FUSE_MEAN writes the mean to all K rows instead of the K different values: the averaging then costs no HBM traffic
// at all, theta is read once and written once exactly as in a plain step.  FUSE_SUM is the multi-GPU form: the
// column's sum goes to p.sum_out (the buffer that is all-reduced over processes) and theta is not written at all,
// since the finish kernel will overwrite every row with the global mean.
//
// EXTRAS selects the build that honours the per-tensor weight-decay table and the clipping factors; the plain build
// (no table, clipping off: every run of the paper's QSR experiments) does not carry their tests in the row loop.

template <int OPT, bool EXT_GRAD>
struct StepOperands {
    static constexpr int kStateSlabs = OPT == QSR_OPT_ADAMW ? 2 : 1;
    static constexpr int kCount = 1 + kStateSlabs + (EXT_GRAD ? 1 : 0);   // slots per row and thread
};

// NEXTNORM (gradient clipping on, gradients generated, plain step): the thread that has just formed a worker's new
// parameters also evaluates that worker's NEXT gradient on them and leaves its sum of squares in shared memory; the
// block folds the K x blockDim values into p.norm_partial, laid out and summed exactly as the stand-alone norm pass
// (column_sqnorm_kernel) does.  The following step then needs no norm pass of its own: the parameters are not read a
// second time, and the extra noise evaluation runs in issue slots the memory-bound step leaves free.
template <int OPT, bool EXT_GRAD, int STAGES, int FUSE, bool EXTRAS, bool NEXTNORM>
__global__ void local_step_kernel(const __grid_constant__ StepParams p)
{
    extern __shared__ float4 ring[];   // [STAGES][operands][blockDim.x], then (NEXTNORM) float [K][blockDim.x]
    constexpr int NOP = StepOperands<OPT, EXT_GRAD>::kCount;
    const int tid = threadIdx.x, bd = blockDim.x;
    const int64_t n_col = (p.P + 3) >> 2;
    const int64_t j = int64_t(blockIdx.x) * bd + tid;      // the grid has one thread per column (see grid_for)
    float *norm_acc = reinterpret_cast<float *>(ring + STAGES * NOP * bd);
    if (j >= n_col) {
        if (!NEXTNORM) return;
        for (int k = 0; k < p.K; ++k) norm_acc[k * bd + tid] = 0.f;     // stays for the block's reduction below
    } else {
        const int64_t i0 = j << 2;
        const float wdv = EXTRAS ? weight_decay_at<OPT>(p, i0) : (OPT == QSR_OPT_SGDM ? p.wd : p.eta_wd);
        if (i0 + 4 <= p.P) {
            float4 lam = make_float4(0.f, 0.f, 0.f, 0.f), ths = lam;
            if (!EXT_GRAD) {
                lam = ld4(p.lambda + i0);
                ths = ld4(p.theta_star + i0);
            }
            auto fetch = [&](int k, int stage) {
                const int64_t e = int64_t(k) * p.stride + i0;
                float4 *slot = ring + (stage * NOP) * bd + tid;
                cp_async16(slot, p.theta + e);
                cp_async16(slot + bd, p.s1 + e);
                if (OPT == QSR_OPT_ADAMW) cp_async16(slot + 2 * bd, p.s2 + e);
                if (EXT_GRAD) cp_async16(slot + (NOP - 1) * bd, p.grads + e);
            };
#pragma unroll
            for (int s = 0; s < STAGES; ++s) {      // fill the ring; one group per row, empty groups keep the count uniform
                if (s < p.K) fetch(s, s);
                cp_async_commit();
            }
            float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
            int stage = 0;
            for (int k = 0; k < p.K; ++k) {
                cp_async_wait_all_but<STAGES - 1>();                 // row k has landed
                const float4 *slot = ring + (stage * NOP) * bd + tid;
                float4 th = slot[0], a = slot[bd], b = make_float4(0.f, 0.f, 0.f, 0.f), g;
                if (OPT == QSR_OPT_ADAMW) b = slot[2 * bd];
                if (EXT_GRAD) g = slot[(NOP - 1) * bd];
                if (k + STAGES < p.K) fetch(k + STAGES, stage);      // the slot is free again: refill it
                cp_async_commit();
                stage = stage + 1 == STAGES ? 0 : stage + 1;
                if (!EXT_GRAD) {
                    const float4 z = noise4(j, p.step, p.worker0 + uint32_t(k), p.round_key);
                    g.x = fmaf(p.sigma, z.x, lam.x * (th.x - ths.x));
                    g.y = fmaf(p.sigma, z.y, lam.y * (th.y - ths.y));
                    g.z = fmaf(p.sigma, z.z, lam.z * (th.z - ths.z));
                    g.w = fmaf(p.sigma, z.w, lam.w * (th.w - ths.w));
                }
                if (EXTRAS && p.clip_coef) {   // gradient clipping: this worker's factor min(1, c / (||g|| + 1e-6))
                    const float cs = __ldg(p.clip_coef + k);
                    g.x *= cs; g.y *= cs; g.z *= cs; g.w *= cs;
                }
                opt_update<OPT>(th.x, a.x, b.x, g.x, p, wdv);
                opt_update<OPT>(th.y, a.y, b.y, g.y, p, wdv);
                opt_update<OPT>(th.z, a.z, b.z, g.z, p, wdv);
                opt_update<OPT>(th.w, a.w, b.w, g.w, p, wdv);
                const int64_t e = int64_t(k) * p.stride + i0;
                if (FUSE != FUSE_NONE) acc = add4(acc, th);
                else st4(p.theta + e, th);
                st4(p.s1 + e, a);
                if (OPT == QSR_OPT_ADAMW) st4(p.s2 + e, b);
                if (NEXTNORM) norm_acc[k * bd + tid] = column_sq(p, j, p.step + 1u, k, th, lam, ths, 4);
            }
            if (FUSE == FUSE_MEAN) {
                // At the power-capped clock the SGD step is close to issue-bound and every instruction of this
                // epilogue shows (the round-end launch ran 7.5 % more instructions than a plain step and took 4-6 %
                // longer on boxes that hold only 1.46 GHz): for K a power of two -- every run configuration -- 1/K is
                // exact and the product equals the quotient bit for bit, and the row pointer advances by addition.
                const float4 mean = (p.K & (p.K - 1)) == 0
                                        ? make_float4(acc.x * p.inv_K, acc.y * p.inv_K, acc.z * p.inv_K, acc.w * p.inv_K)
                                        : div4(acc, float(p.K));
                float *row = p.theta + i0;
#pragma unroll 4
                for (int k = 0; k < p.K; ++k) {
                    st4(row, mean);
                    row += p.stride;
                }
            } else if (FUSE == FUSE_SUM) {
                st4(p.sum_out + i0, acc);
            }
        } else {
            // Ragged last column: P is not a multiple of 4.  Scalar accesses, nothing beyond P is touched.
            for (int64_t i = i0; i < p.P; ++i) {
                const int c = int(i - i0);                                  // 0, 1 or 2
                float acc = 0.f;
                for (int k = 0; k < p.K; ++k) {
                    const int64_t e = int64_t(k) * p.stride + i;
                    float th = p.theta[e], a = p.s1[e], b = OPT == QSR_OPT_ADAMW ? p.s2[e] : 0.f;
                    float g;
                    if (EXT_GRAD) {
                        g = p.grads[e];
                    } else {
                        const float4 z = noise4(j, p.step, p.worker0 + uint32_t(k), p.round_key);
                        const float zc = c == 0 ? z.x : (c == 1 ? z.y : z.z);
                        g = fmaf(p.sigma, zc, p.lambda[i] * (th - p.theta_star[i]));
                    }
                    if (EXTRAS && p.clip_coef) g *= __ldg(p.clip_coef + k);
                    opt_update<OPT>(th, a, b, g, p, wdv);
                    if (FUSE != FUSE_NONE) acc += th;
                    else p.theta[e] = th;
                    p.s1[e] = a;
                    if (OPT == QSR_OPT_ADAMW) p.s2[e] = b;
                }
                if (FUSE == FUSE_MEAN) {
                    const float mean = acc / float(p.K);
                    for (int k = 0; k < p.K; ++k) p.theta[int64_t(k) * p.stride + i] = mean;
                } else if (FUSE == FUSE_SUM) {
                    p.sum_out[i] = acc;
                }
            }
            if (NEXTNORM) {            // the ragged column's share of the next norms, from the values just written
                const int valid = int(p.P - i0);
                const float4 lam = ld4_guarded(p.lambda + i0, valid), ths = ld4_guarded(p.theta_star + i0, valid);
                for (int k = 0; k < p.K; ++k)
                    norm_acc[k * bd + tid] = column_sq(p, j, p.step + 1u, k, ld4_guarded(p.theta + int64_t(k) * p.stride + i0, valid),
                                                       lam, ths, valid);
            }
        }
    }
    if (NEXTNORM) {
        __syncthreads();
        reduce_rows_to_partials(norm_acc, p.K, p.norm_partial);
    }
}

// Sum over rows of one 16-byte column, k ascending, eight loads in flight.
__device__ __forceinline__ float4 column_sum(const float *slab, int64_t i0, int64_t stride, int K)
{
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    int k = 0;
    for (; k + 8 <= K; k += 8) {
        float4 v[8];
#pragma unroll
        for (int r = 0; r < 8; ++r) v[r] = ld4(slab + int64_t(k + r) * stride + i0);
#pragma unroll
        for (int r = 0; r < 8; ++r) acc = add4(acc, v[r]);
    }
    for (; k < K; ++k) acc = add4(acc, ld4(slab + int64_t(k) * stride + i0));
    return acc;
}

// ---------------------------------------------------------------------------------------------- Algorithm 1

// Parallel OPT: the single model lives in row 0 of the slabs; the K workers' gradients are all taken at that one
// point, summed for k = 0..K-1 and divided by K (the All-Reduce line of Algorithm 1), and one optimizer step follows.
// HBM traffic is that of one row (plus the K gradient rows when they come from a slab); with generated gradients the
// kernel is bound by the K noise evaluations per coordinate, not by memory.
template <int OPT, bool EXT_GRAD>
__global__ void parallel_step_kernel(const __grid_constant__ StepParams p)
{
    const int64_t n_col = (p.P + 3) >> 2;
    const int64_t grid_stride = int64_t(gridDim.x) * blockDim.x;
    const float Kf = float(p.K);
    for (int64_t j = int64_t(blockIdx.x) * blockDim.x + threadIdx.x; j < n_col; j += grid_stride) {
        const int64_t i0 = j << 2;
        const float wdv = weight_decay_at<OPT>(p, i0);
        if (i0 + 4 <= p.P) {
            float4 th = ld4(p.theta + i0), a = ld4(p.s1 + i0), b = make_float4(0.f, 0.f, 0.f, 0.f);
            if (OPT == QSR_OPT_ADAMW) b = ld4(p.s2 + i0);
            float4 sum = make_float4(0.f, 0.f, 0.f, 0.f);
            if (EXT_GRAD) {
                sum = column_sum(p.grads, i0, p.stride, p.K);
            } else {
                const float4 lam = ld4(p.lambda + i0), ths = ld4(p.theta_star + i0);
                const float4 pull = make_float4(lam.x * (th.x - ths.x), lam.y * (th.y - ths.y),
                                                lam.z * (th.z - ths.z), lam.w * (th.w - ths.w));
                for (int k = 0; k < p.K; ++k) {
                    const float4 z = noise4_packed(j, p.step, p.worker0 + uint32_t(k), p.round_key);
                    const float2 lo = add2(make_float2(sum.x, sum.y),
                                           fma2(both(p.sigma), make_float2(z.x, z.y), make_float2(pull.x, pull.y)));
                    const float2 hi = add2(make_float2(sum.z, sum.w),
                                           fma2(both(p.sigma), make_float2(z.z, z.w), make_float2(pull.z, pull.w)));
                    sum = make_float4(lo.x, lo.y, hi.x, hi.y);
                }
            }
            float4 g = div4(sum, Kf);
            if (p.clip_coef) {   // clipping acts on the averaged gradient
                const float cs = __ldg(p.clip_coef);
                g.x *= cs; g.y *= cs; g.z *= cs; g.w *= cs;
            }
            opt_update4<OPT>(th, a, b, g, p, wdv);
            st4(p.theta + i0, th);
            st4(p.s1 + i0, a);
            if (OPT == QSR_OPT_ADAMW) st4(p.s2 + i0, b);
        } else {
            for (int64_t i = i0; i < p.P; ++i) {
                const int c = int(i - i0);
                float th = p.theta[i], a = p.s1[i], b = OPT == QSR_OPT_ADAMW ? p.s2[i] : 0.f;
                float sum = 0.f;
                for (int k = 0; k < p.K; ++k) {
                    if (EXT_GRAD) {
                        sum += p.grads[int64_t(k) * p.stride + i];
                    } else {
                        const float4 z = noise4(j, p.step, p.worker0 + uint32_t(k), p.round_key);
                        const float zc = c == 0 ? z.x : (c == 1 ? z.y : z.z);
                        sum += fmaf(p.sigma, zc, p.lambda[i] * (th - p.theta_star[i]));
                    }
                }
                float g = sum / Kf;
                if (p.clip_coef) g *= __ldg(p.clip_coef);
                opt_update<OPT>(th, a, b, g, p, wdv);
                p.theta[i] = th;
                p.s1[i] = a;
                if (OPT == QSR_OPT_ADAMW) p.s2[i] = b;
            }
        }
    }
}

// ---------------------------------------------------------------------------------------------- gradient clipping

// Pass 1 of global-norm clipping (App. C.2) for Local OPT: per worker k the sum of squares of the gradient its step
// will use, as partial sums per block.  Generated gradients are recomputed here with the very expressions of the step
// kernel -- the noise is a pure function of (seed, worker, step, coordinate) -- so nothing has to be stored: the pass
// reads theta once (4 B per update).  The geometry is the step kernel's (one thread per column, the step's block
// size) and the per-column value and the block's reduction are shared code, so the partials equal, bit for bit, what a
// step launched with NEXTNORM leaves behind for its successor.  partial is [gridDim.x, K].
template <bool EXT_GRAD>
__global__ void column_sqnorm_kernel(const __grid_constant__ StepParams p, float *partial)
{
    extern __shared__ float norm_acc[];     // [K][blockDim.x]
    const int tid = threadIdx.x, bd = blockDim.x;
    const int64_t n_col = (p.P + 3) >> 2;
    const int64_t j = int64_t(blockIdx.x) * bd + tid;
    if (j < n_col) {
        const int64_t i0 = j << 2;
        const int valid = i0 + 4 <= p.P ? 4 : int(p.P - i0);
        float4 lam = make_float4(0.f, 0.f, 0.f, 0.f), ths = lam;
        if (!EXT_GRAD) {
            lam = ld4_guarded(p.lambda + i0, valid);
            ths = ld4_guarded(p.theta_star + i0, valid);
        }
        const float *src = EXT_GRAD ? p.grads : p.theta;
        auto one_row = [&](int k, float4 v) {
            if (EXT_GRAD) norm_acc[k * bd + tid] = fmaf(v.x, v.x, v.y * v.y) + fmaf(v.z, v.z, v.w * v.w);   // zeros beyond P
            else norm_acc[k * bd + tid] = column_sq(p, j, p.step, k, v, lam, ths, valid);
        };
        int k = 0;
        for (; k + 4 <= p.K; k += 4) {      // four rows' loads in flight before the arithmetic of the first
            float4 v[4];
#pragma unroll
            for (int r = 0; r < 4; ++r) v[r] = ld4_guarded(src + int64_t(k + r) * p.stride + i0, valid);
#pragma unroll
            for (int r = 0; r < 4; ++r) one_row(k + r, v[r]);
        }
        for (; k < p.K; ++k) one_row(k, ld4_guarded(src + int64_t(k) * p.stride + i0, valid));
    } else {
        for (int k = 0; k < p.K; ++k) norm_acc[k * bd + tid] = 0.f;
    }
    __syncthreads();
    reduce_rows_to_partials(norm_acc, p.K, partial);
}

// The same pass for Algorithm 1: the squared norm of the AVERAGED gradient, all K gradients taken at the single model
// in row 0.  The grid is fixed (kNormGrid blocks at most); a thread strides over columns and keeps a running sum.
// partial is [gridDim.x].  Summation order is fixed: results are deterministic.
template <bool EXT_GRAD>
__global__ void parallel_sqnorm_kernel(const __grid_constant__ StepParams p, float *partial)
{
    extern __shared__ float acc[];
    acc[threadIdx.x] = 0.f;
    const int64_t n_col = (p.P + 3) >> 2;
    const int64_t grid_stride = int64_t(gridDim.x) * blockDim.x;
    const float Kf = float(p.K);
    for (int64_t j = int64_t(blockIdx.x) * blockDim.x + threadIdx.x; j < n_col; j += grid_stride) {
        const int64_t i0 = j << 2;
        const int valid = i0 + 4 <= p.P ? 4 : int(p.P - i0);
        float4 lam = make_float4(0.f, 0.f, 0.f, 0.f), ths = lam, sum = lam, th = lam;
        if (!EXT_GRAD) {
            lam = ld4_guarded(p.lambda + i0, valid);     // zero lambda and zero noise weight make the lanes beyond P vanish
            ths = ld4_guarded(p.theta_star + i0, valid);
            th = ld4_guarded(p.theta + i0, valid);
        }
        for (int k = 0; k < p.K; ++k) {
            float4 g;
            if (EXT_GRAD) {
                g = ld4_guarded(p.grads + int64_t(k) * p.stride + i0, valid);
            } else {
                const float4 z = noise4_packed(j, p.step, p.worker0 + uint32_t(k), p.round_key);
                g = gradient4(p.sigma, z, lam, th, ths);
                if (valid < 4) {                   // ragged last column: the lanes beyond P do not count
                    g.y = valid > 1 ? g.y : 0.f;
                    g.z = valid > 2 ? g.z : 0.f;
                    g.w = 0.f;
                }
            }
            sum = add4(sum, g);
        }
        sum = div4(sum, Kf);
        acc[threadIdx.x] += (sum.x * sum.x + sum.y * sum.y) + (sum.z * sum.z + sum.w * sum.w);
    }
    __syncthreads();
    reduce_rows_to_partials(acc, 1, partial);
}

// Pass 2: coef[r] = min(1, max_norm / (sqrt(sum of partials) + 1e-6)).  One block per row; every thread adds its
// stride of the row's partials in binary64, then the block folds the 256 sums in a fixed tree: deterministic.
__global__ void __launch_bounds__(256) clip_coef_kernel(const float *partial, int64_t n_blocks, int rows, double max_norm,
                                                         float *coef)
{
    __shared__ double part[256];
    const int r = blockIdx.x;
    double s = 0.0;
    for (int64_t b = threadIdx.x; b < n_blocks; b += 256) s += double(partial[b * rows + r]);
    part[threadIdx.x] = s;
    __syncthreads();
    for (int o = 128; o; o >>= 1) {
        if (int(threadIdx.x) < o) part[threadIdx.x] += part[threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        const double c = max_norm / (sqrt(part[0]) + 1e-6);
        coef[r] = float(c < 1.0 ? c : 1.0);
    }
}

// ---------------------------------------------------------------------------------------------- synchronization

// One array's share of a synchronization for the column (or ragged tail) that starts at coordinate i0.
// MODE 0: mean of the rows, written back to every row (the whole synchronization on one GPU).
// MODE 1: sums only, written to sum_out (first half of a synchronization sharded over GPUs).
// MODE 2: rows <- sum_in / divisor (second half).
template <int MODE>
__device__ __forceinline__ void sync_column(float *slab, const float *sum_in, float *sum_out, int64_t i0,
                                            const SyncParams &p)
{
    if (i0 + 4 <= p.P) {
        float4 s;
        if (MODE == 2) s = ld4(sum_in + i0);
        else s = column_sum(slab, i0, p.stride, p.K);
        if (MODE == 1) {
            st4(sum_out + i0, s);
        } else {
            const float4 mean = div4(s, p.divisor);
#pragma unroll 4
            for (int k = 0; k < p.K; ++k) st4(slab + int64_t(k) * p.stride + i0, mean);
        }
    } else {
        for (int64_t i = i0; i < p.P; ++i) {
            float s = 0.f;
            if (MODE == 2) s = sum_in[i];
            else for (int k = 0; k < p.K; ++k) s += slab[int64_t(k) * p.stride + i];
            if (MODE == 1) {
                sum_out[i] = s;
            } else {
                const float mean = s / p.divisor;
                for (int k = 0; k < p.K; ++k) slab[int64_t(k) * p.stride + i] = mean;
            }
        }
    }
}

// slab[0 .. n_mean) are averaged (theta always; the optimizer state in AVERAGE mode).  A thread owns one 16-byte
// column of all K rows: eight row loads in flight, the sum in registers, one division, K stores.  The second half of
// a sharded synchronization (MODE 2) keeps this shape although it only reads one vector: the division is then done
// once per column, where one-row-per-block would repeat it for each of the K rows and become bound by it.
template <int MODE>
__global__ void __launch_bounds__(512) sync_kernel(const SyncParams p)
{
    const int64_t n_col = (p.P + 3) >> 2;
    const int64_t grid_stride = int64_t(gridDim.x) * blockDim.x;
    for (int64_t j = int64_t(blockIdx.x) * blockDim.x + threadIdx.x; j < n_col; j += grid_stride) {
        const int64_t i0 = j << 2;
#pragma unroll
        for (int a = 0; a < 3; ++a)
            if (a < p.n_mean) sync_column<MODE>(p.slab[a], p.sum_in + a * p.P4, p.sum_out + a * p.P4, i0, p);
    }
}

// Rows written with zeros or from one source vector: the reset of the optimizer state and the replica copy of the
// initial parameters.  These launches write K times what they read (or read nothing), and a write-only stream runs
// at its best rate when it is not interleaved with a thread's own loads: B200 fills K rows of the ViT-B/16 set at
// 7.3 TB/s from blocks that each write one contiguous 16 KB piece of one row, against 6.1 TB/s for the same zeros
// stored by the threads of the averaging kernel after their K loads, and the one-to-K copy gains 4 % in this form
// over one-column-per-thread.
// Work item = (piece of kRowPiece columns, row); the K rows of a piece are neighbouring items, so the K blocks that
// need the same piece of the source run together and all but the first find it in L2.
constexpr int kRowThreads = 256, kRowColsPerThread = 4, kRowPiece = kRowThreads * kRowColsPerThread;

struct RowsParams {
    float *dst[3];            // up to three slabs [K, stride]
    const float *src[3];      // source vector [P] of each slab (SRC 1)
    int32_t n_slabs, K;
    int64_t P, stride;
};

// SRC 0: zeros.  SRC 1: copy of src.
template <int SRC>
__global__ void __launch_bounds__(kRowThreads) rows_kernel(const __grid_constant__ RowsParams p)
{
    const int64_t n_col = (p.P + 3) >> 2;
    const int64_t pieces = (n_col + kRowPiece - 1) / kRowPiece;
    const int64_t rows = int64_t(p.n_slabs) * p.K;
    const int64_t items = pieces * rows;
    for (int64_t item = blockIdx.x; item < items; item += gridDim.x) {
        const int64_t piece = item / rows;
        const int r = int(item - piece * rows);
        const int a = r / p.K, k = r - a * p.K;
        float *row = p.dst[a] + int64_t(k) * p.stride;
        const float *src = p.src[a];
        const int64_t j0 = piece * kRowPiece + threadIdx.x;
        float4 v[kRowColsPerThread];
#pragma unroll
        for (int c = 0; c < kRowColsPerThread; ++c) {
            const int64_t i0 = (j0 + int64_t(c) * kRowThreads) << 2;
            v[c] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (SRC != 0 && i0 + 4 <= p.P) v[c] = ld4(src + i0);
        }
#pragma unroll
        for (int c = 0; c < kRowColsPerThread; ++c) {
            const int64_t i0 = (j0 + int64_t(c) * kRowThreads) << 2;
            if (i0 + 4 <= p.P) st4(row + i0, v[c]);
        }
        // Ragged end of the row (P not a multiple of 4): its one to three floats are written, one per thread, by the
        // block that holds the row's last piece.  Kept out of the loops above, whose four loads and four stores the
        // compiler otherwise no longer issues back to back (10 % on the one-to-K copy).
        if (piece == pieces - 1 && int(threadIdx.x) < int(p.P & 3)) {
            const int64_t i = (p.P & ~int64_t(3)) + threadIdx.x;
            row[i] = SRC == 0 ? 0.f : src[i];
        }
    }
}

template <int SRC>
int launch_rows(const RowsParams &p, void *stream)
{
    const int64_t n_col = (p.P + 3) >> 2;
    int64_t items = ((n_col + kRowPiece - 1) / kRowPiece) * int64_t(p.n_slabs) * p.K;
    if (items > 2147483647) items = 2147483647;     // the kernel strides over the rest
    if (items < 1) return 0;
    rows_kernel<SRC><<<unsigned(items), kRowThreads, 0, static_cast<cudaStream_t>(stream)>>>(p);
    return int(cudaGetLastError());
}

// ---------------------------------------------------------------------------------------------- resident steps
//
// q.n_steps consecutive local steps of Algorithm 2's inner loop in one launch.  A thread owns ONE row of one 16-byte
// column: the rows of a column are independent between synchronizations, so spreading them over threads keeps the
// register count low (theta, the state and lambda / theta* of four coordinates) and the machine full even when the
// whole problem is a megabyte.  The block holds all K rows of its 32 (or 64) columns -- thread = row * columns +
// column, so a warp still reads 512 contiguous bytes of one row -- and that makes the averaging block-local: where a
// step ends a round (bit h of q.sync_after) the rows' new parameters go through shared memory and every thread forms
// the mean itself, k ascending from zero and one division, i.e. the bits of the fused last step of the per-step path.
// A launch can therefore run across round ends.  Slabs are read once at the start and written once at the end:
// the launch is bound by the instruction stream of the noise generator and the optimizer, not by memory.
// The arithmetic of a step is the per-step kernel's (same device functions, same expressions): results are
// bit-identical to n_steps single launches.
template <int OPT>
__global__ void resident_steps_kernel(const __grid_constant__ ResidentParams q)
{
    extern __shared__ float4 round_end[];      // [K][cols_per_block]
    const StepParams &p = q.base;
    const int cx = q.cols_per_block;
    const int c = int(threadIdx.x) % cx, k = int(threadIdx.x) / cx;
    const int64_t n_col = (p.P + 3) >> 2;
    const int64_t j = int64_t(blockIdx.x) * cx + c;
    const int64_t i0 = j << 2;
    // threads past the last column stay in the loop for the barriers; they load and store nothing
    const int valid = j < n_col ? (i0 + 4 <= p.P ? 4 : int(p.P - i0)) : 0;
    const int64_t e = int64_t(k) * p.stride + i0;
    const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);
    float4 th = zero, a = zero, b = zero, lam = zero, ths = zero;
    if (valid == 4) {
        th = ld4(p.theta + e);
        a = ld4(p.s1 + e);
        if (OPT == QSR_OPT_ADAMW) b = ld4(p.s2 + e);
        lam = ld4(p.lambda + i0);
        ths = ld4(p.theta_star + i0);
    } else if (valid > 0) {
        th = ld4_guarded(p.theta + e, valid);
        a = ld4_guarded(p.s1 + e, valid);
        if (OPT == QSR_OPT_ADAMW) b = ld4_guarded(p.s2 + e, valid);
        lam = ld4_guarded(p.lambda + i0, valid);
        ths = ld4_guarded(p.theta_star + i0, valid);
    }
    StepParams s;                              // the scalars opt_update reads; everything else stays unused
    s.mu = p.mu; s.omb1 = p.omb1; s.omb2 = p.omb2; s.eps = p.eps;
    const float Kf = float(p.K);
    for (int h = 0; h < q.n_steps; ++h) {
        const ResidentScalars sc = q.per_step[h];
        s.eta = sc.eta; s.step_size = sc.step_size; s.inv_sqrt_bc2 = sc.inv_sqrt_bc2;
        const float wdv = OPT == QSR_OPT_SGDM ? p.wd : sc.eta_wd;
        const float4 z = noise4_packed(j, p.step + uint32_t(h), p.worker0 + uint32_t(k), p.round_key);
        const float4 g = gradient4(p.sigma, z, lam, th, ths);
        opt_update4<OPT>(th, a, b, g, s, wdv);
        if ((q.sync_after[h >> 5] >> (h & 31)) & 1u) {      // uniform over the grid: every thread takes the barriers
            round_end[k * cx + c] = th;
            __syncthreads();
            float4 acc = zero;
            for (int r = 0; r < p.K; ++r) acc = add4(acc, round_end[r * cx + c]);
            th = div4(acc, Kf);
            __syncthreads();
        }
    }
    if (valid == 4) {
        st4(p.theta + e, th);
        st4(p.s1 + e, a);
        if (OPT == QSR_OPT_ADAMW) st4(p.s2 + e, b);
    } else if (valid > 0) {
        for (int l = 0; l < valid; ++l) {          // ragged last column: lanes 0 .. valid-1 (at most three)
            p.theta[e + l] = l == 0 ? th.x : (l == 1 ? th.y : th.z);
            p.s1[e + l] = l == 0 ? a.x : (l == 1 ? a.y : a.z);
            if (OPT == QSR_OPT_ADAMW) p.s2[e + l] = l == 0 ? b.x : (l == 1 ? b.y : b.z);
        }
    }
}

// ---------------------------------------------------------------------------------------------- test hook
//
// The two halves of the Box-Muller transform for a list of generator words, through the very device functions the
// step kernels inline (neg2_log_unit, sqrt_fast, sincos_turn_bits): word w gives the radius sqrt(-2 ln u) for
// u = (w >> 9 + 1/2) / 2^23 and the sine / cosine of the angle 2 pi u.  The grid of inputs has only 2^23 points, so a
// test can walk all of it and bound the error of each part against binary64.
__global__ void box_muller_parts_kernel(const uint32_t *words, int64_t n, float *radius, float *sine, float *cosine)
{
    const int64_t grid_stride = int64_t(gridDim.x) * blockDim.x;
    for (int64_t i = int64_t(blockIdx.x) * blockDim.x + threadIdx.x; i < n; i += grid_stride) {
        const uint32_t w = words[i];
        float s, c;
        sincos_turn_bits(w, s, c);
        radius[i] = sqrt_fast(neg2_log_unit(w));
        sine[i] = s;
        cosine[i] = c;
    }
}

// The two single-instruction special functions of the optimizer update (sqrt_fast for AdamW's root of the second
// moment and the Box-Muller radius, rcp_fast for AdamW's quotient), for tests that bound their error.
__global__ void fast_math_kernel(const float *x, int64_t n, float *root, float *reciprocal)
{
    const int64_t grid_stride = int64_t(gridDim.x) * blockDim.x;
    for (int64_t i = int64_t(blockIdx.x) * blockDim.x + threadIdx.x; i < n; i += grid_stride) {
        root[i] = sqrt_fast(x[i]);
        reciprocal[i] = rcp_fast(x[i]);
    }
}

// One thread per 16-byte column.  2^31 - 1 blocks of at least 64 threads cover rows of 2^39 floats, beyond any device
// memory, so the kernels that rely on full coverage (local_step_kernel) never meet a capped grid.
unsigned grid_for(int64_t P, int threads)
{
    const int64_t n_col = (P + 3) >> 2;
    int64_t blocks = (n_col + threads - 1) / threads;
    const int64_t cap = 2147483647;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    return unsigned(blocks);
}

// Picks one instance of the step kernel and its launch geometry; raises the instance's dynamic shared-memory limit
// (the ring exceeds the 48 KB default).  Returns a cudaError_t as int.
template <int OPT, bool EXT, int STAGES, int FUSE, bool EXTRAS, bool NEXTNORM>
int resolve_step_instance(const StepParams &p, int threads, StepLaunch *out)
{
    const size_t smem = step_shared_bytes(OPT, EXT, STAGES, threads, NEXTNORM ? p.K : 0);
    if (smem > 227 * 1024) return int(cudaErrorInvalidValue);
    auto kernel = local_step_kernel<OPT, EXT, STAGES, FUSE, EXTRAS, NEXTNORM>;
    if (smem > 48 * 1024) {
        if (cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem)))
            return int(e);
    }
    out->func = reinterpret_cast<const void *>(kernel);
    out->grid = grid_for(p.P, threads);
    out->threads = threads;
    out->smem = smem;
    return 0;
}

template <int OPT, bool EXT, int FUSE, bool EXTRAS, bool NEXTNORM>
int resolve_step_stages(const StepParams &p, const LaunchShape &s, StepLaunch *out)
{
    switch (s.step_rows ? s.step_rows : 8) {
    case 1: return resolve_step_instance<OPT, EXT, 1, FUSE, EXTRAS, NEXTNORM>(p, s.step_threads, out);
    case 2: return resolve_step_instance<OPT, EXT, 2, FUSE, EXTRAS, NEXTNORM>(p, s.step_threads, out);
    case 4: return resolve_step_instance<OPT, EXT, 4, FUSE, EXTRAS, NEXTNORM>(p, s.step_threads, out);
    default: return resolve_step_instance<OPT, EXT, 8, FUSE, EXTRAS, NEXTNORM>(p, s.step_threads, out);
    }
}

template <int OPT, bool EXT, int FUSE>
int resolve_step_extras(const StepParams &p, const LaunchShape &s, StepLaunch *out)
{
    if (p.norm_partial) {       // only the plain step with generated gradients computes the next norms on the side
        if (EXT || FUSE != FUSE_NONE) return int(cudaErrorInvalidValue);
        return resolve_step_stages<OPT, false, FUSE_NONE, true, true>(p, s, out);
    }
    if (p.n_tensors > 0 || p.clip_coef) return resolve_step_stages<OPT, EXT, FUSE, true, false>(p, s, out);
    return resolve_step_stages<OPT, EXT, FUSE, false, false>(p, s, out);
}

template <int FUSE>
int resolve_step_fuse(const StepParams &p, int opt, const LaunchShape &shape, StepLaunch *out)
{
    const bool ext = p.grads != nullptr;
    if (opt == QSR_OPT_SGDM)
        return ext ? resolve_step_extras<QSR_OPT_SGDM, true, FUSE>(p, shape, out)
                   : resolve_step_extras<QSR_OPT_SGDM, false, FUSE>(p, shape, out);
    return ext ? resolve_step_extras<QSR_OPT_ADAMW, true, FUSE>(p, shape, out)
               : resolve_step_extras<QSR_OPT_ADAMW, false, FUSE>(p, shape, out);
}

int launch_resolved(const StepParams &p, int opt, const LaunchShape &shape, int fuse, void *stream)
{
    StepLaunch L;
    if (int rc = resolve_step(p, opt, shape, fuse, &L)) return rc;
    void *args[] = {const_cast<StepParams *>(&p)};
    return int(cudaLaunchKernel(L.func, dim3(L.grid), dim3(unsigned(L.threads)), args, L.smem,
                                static_cast<cudaStream_t>(stream)));
}

}  // namespace

// Dynamic shared memory of a step launch: the ring, plus K x threads floats when the next step's norms ride along.
size_t step_shared_bytes(int opt, bool ext_grad, int stages, int threads, int next_norm_rows)
{
    const int operands = 1 + (opt == QSR_OPT_ADAMW ? 2 : 1) + (ext_grad ? 1 : 0);
    return size_t(stages) * operands * threads * sizeof(float4) + size_t(next_norm_rows) * threads * sizeof(float);
}

int resolve_step(const StepParams &p, int opt, const LaunchShape &shape, int fuse, StepLaunch *out)
{
    switch (fuse) {
    case FUSE_NONE: return resolve_step_fuse<FUSE_NONE>(p, opt, shape, out);
    case FUSE_MEAN: return resolve_step_fuse<FUSE_MEAN>(p, opt, shape, out);
    case FUSE_SUM: return resolve_step_fuse<FUSE_SUM>(p, opt, shape, out);
    default: return int(cudaErrorInvalidValue);
    }
}

int launch_step(const StepParams &p, int opt, const LaunchShape &shape, void *stream)
{
    return launch_resolved(p, opt, shape, FUSE_NONE, stream);
}

int launch_step_mean(const StepParams &p, int opt, const LaunchShape &shape, void *stream)
{
    return launch_resolved(p, opt, shape, FUSE_MEAN, stream);
}

int launch_step_sum(const StepParams &p, int opt, const LaunchShape &shape, void *stream)
{
    return launch_resolved(p, opt, shape, FUSE_SUM, stream);
}

int launch_parallel_step(const StepParams &p, int opt, const LaunchShape &shape, void *stream)
{
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const unsigned grid = grid_for(p.P, shape.step_threads);
    const bool ext = p.grads != nullptr;
    if (opt == QSR_OPT_SGDM) {
        if (ext) parallel_step_kernel<QSR_OPT_SGDM, true><<<grid, shape.step_threads, 0, st>>>(p);
        else parallel_step_kernel<QSR_OPT_SGDM, false><<<grid, shape.step_threads, 0, st>>>(p);
    } else {
        if (ext) parallel_step_kernel<QSR_OPT_ADAMW, true><<<grid, shape.step_threads, 0, st>>>(p);
        else parallel_step_kernel<QSR_OPT_ADAMW, false><<<grid, shape.step_threads, 0, st>>>(p);
    }
    return int(cudaGetLastError());
}

int clip_grid(int64_t P)
{
    const int64_t want = (((P + 3) >> 2) + kNormThreads - 1) / kNormThreads;
    return int(want < kNormGrid ? (want < 1 ? 1 : want) : kNormGrid);
}

// Blocks of the per-worker norm pass = blocks of a step launch with this block size: one thread per column.
int64_t clip_norm_blocks(int64_t P, int threads) { return int64_t(grid_for(P, threads)); }

// Enqueues the norm pass of Local OPT: ws[0 .. blocks * K) receives the partial sums.
int launch_clip_norms(const StepParams &p, float *ws, const LaunchShape &shape, void *stream)
{
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int threads = shape.step_threads;
    const size_t smem = size_t(p.K) * threads * sizeof(float);
    if (smem > 227 * 1024) return int(cudaErrorInvalidValue);
    auto kernel = p.grads ? column_sqnorm_kernel<true> : column_sqnorm_kernel<false>;
    if (smem > 48 * 1024)
        if (cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem))) return int(e);
    kernel<<<grid_for(p.P, threads), threads, smem, st>>>(p, ws);
    return int(cudaGetLastError());
}

// Enqueues the factor pass over `blocks` partials per row: ws[blocks * rows .. +rows) receives the factors.
int launch_clip_factors(float *ws, int64_t blocks, int rows, double max_norm, void *stream)
{
    clip_coef_kernel<<<unsigned(rows), 256, 0, static_cast<cudaStream_t>(stream)>>>(ws, blocks, rows, max_norm, ws + blocks * rows);
    return int(cudaGetLastError());
}

// Algorithm 1: both clipping passes; afterwards ws[clip_grid(P)] holds the factor.
int launch_clip_coef_parallel(const StepParams &p, double max_norm, float *ws, void *stream)
{
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int grid = clip_grid(p.P);
    const size_t smem = size_t(kNormThreads) * sizeof(float);
    if (p.grads) parallel_sqnorm_kernel<true><<<grid, kNormThreads, smem, st>>>(p, ws);
    else parallel_sqnorm_kernel<false><<<grid, kNormThreads, smem, st>>>(p, ws);
    if (cudaError_t e = cudaGetLastError()) return int(e);
    return launch_clip_factors(ws, grid, 1, max_norm, stream);
}

// The state slabs a synchronization resets: a launch of its own after the averaging (see rows_kernel).
static int launch_state_reset(const SyncParams &p, void *stream)
{
    if (p.n_zero == 0) return 0;
    RowsParams r;
    std::memset(&r, 0, sizeof r);
    for (int a = 0; a < p.n_zero; ++a) r.dst[a] = p.slab[p.n_mean + a];
    r.n_slabs = p.n_zero; r.K = p.K; r.P = p.P; r.stride = p.stride;
    return launch_rows<0>(r, stream);
}

int launch_sync(const SyncParams &p, const LaunchShape &shape, void *stream)
{
    sync_kernel<0><<<grid_for(p.P, shape.sync_threads), shape.sync_threads, 0, static_cast<cudaStream_t>(stream)>>>(p);
    if (cudaError_t e = cudaGetLastError()) return int(e);
    return launch_state_reset(p, stream);
}

int launch_sync_partial(const SyncParams &p, const LaunchShape &shape, void *stream)
{
    sync_kernel<1><<<grid_for(p.P, shape.sync_threads), shape.sync_threads, 0, static_cast<cudaStream_t>(stream)>>>(p);
    return int(cudaGetLastError());
}

int launch_sync_finish(const SyncParams &p, const LaunchShape &shape, void *stream)
{
    sync_kernel<2><<<grid_for(p.P, shape.sync_threads), shape.sync_threads, 0, static_cast<cudaStream_t>(stream)>>>(p);
    if (cudaError_t e = cudaGetLastError()) return int(e);
    return launch_state_reset(p, stream);
}

int launch_broadcast(float *theta, const float *theta0, int64_t P, int64_t stride, int32_t K,
                     const LaunchShape &shape, void *stream)
{
    RowsParams r;
    std::memset(&r, 0, sizeof r);
    r.dst[0] = theta; r.src[0] = theta0;
    r.n_slabs = 1; r.K = K; r.P = P; r.stride = stride;
    return launch_rows<1>(r, stream);
}

int launch_resident_steps(const ResidentParams &q, int opt, void *stream)
{
    const int64_t n_col = (q.base.P + 3) >> 2;
    const int cx = q.cols_per_block;
    const int64_t blocks = (n_col + cx - 1) / cx;
    if (blocks > 2147483647 || q.base.K > kMaxResidentK || cx * q.base.K > 1024) return int(cudaErrorInvalidValue);
    const unsigned threads = unsigned(cx * q.base.K);
    const size_t smem = size_t(threads) * sizeof(float4);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (opt == QSR_OPT_SGDM) resident_steps_kernel<QSR_OPT_SGDM><<<unsigned(blocks), threads, smem, st>>>(q);
    else resident_steps_kernel<QSR_OPT_ADAMW><<<unsigned(blocks), threads, smem, st>>>(q);
    return int(cudaGetLastError());
}

int launch_fast_math(const float *x, int64_t n, float *root, float *reciprocal, void *stream)
{
    int64_t blocks = (n + 255) / 256;
    if (blocks > 148 * 16) blocks = 148 * 16;
    if (blocks < 1) blocks = 1;
    fast_math_kernel<<<unsigned(blocks), 256, 0, static_cast<cudaStream_t>(stream)>>>(x, n, root, reciprocal);
    return int(cudaGetLastError());
}

int launch_box_muller_parts(const uint32_t *words, int64_t n, float *radius, float *sine, float *cosine, void *stream)
{
    int64_t blocks = (n + 255) / 256;
    if (blocks > 148 * 16) blocks = 148 * 16;
    if (blocks < 1) blocks = 1;
    box_muller_parts_kernel<<<unsigned(blocks), 256, 0, static_cast<cudaStream_t>(stream)>>>(words, n, radius, sine, cosine);
    return int(cudaGetLastError());
}

}  // namespace qsr

// ---------------------------------------------------------------------------------------------- static scratch
//
// Scratch of the two-phase synchronization for callers that cannot hand the library a buffer of their own.  It lives
// in the library image: every GPU that loads the library holds these 4 MiB until the process exits.  In host code the
// name `g_sync_scratch` is only a handle for the runtime; the address a kernel can use is the one
// cudaGetSymbolAddress returns for the device that is current at the time.
static __device__ __align__(256) float g_sync_scratch[QSR_STATIC_SCRATCH_FLOATS];

namespace qsr {

namespace {
constexpr int kMaxDevices = 64;
// Device address of g_sync_scratch per device ordinal (null = not yet asked).  Atomic, so that contexts on different
// host threads may make their first call at the same time: both look the same address up and store the same value.
std::atomic<float *> g_scratch_addr[kMaxDevices];
}  // namespace

// The two phases (row sums into the static array, then rows <- sums / K) enqueued back to back on `stream`.
// `device` is the ordinal the context was created on; it must be the current one, because the array's address is
// looked up for the current device.  Returns 0, a cudaError_t, -1 when the sums do not fit, -2 when another device
// is current.  The first call on a device looks the array's device address up; no memory is allocated or freed here.
int launch_sync_static(const SyncParams &p_in, const LaunchShape &shape, int device, void *stream)
{
    if (int64_t(p_in.n_mean) * p_in.P4 > int64_t(QSR_STATIC_SCRATCH_FLOATS)) return -1;
    int dev = -1;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return int(err);
    if (dev != device) return -2;
    if (dev < 0 || dev >= kMaxDevices) return int(cudaErrorInvalidDevice);
    float *scratch = g_scratch_addr[dev].load(std::memory_order_acquire);
    if (!scratch) {
        err = cudaGetSymbolAddress(reinterpret_cast<void **>(&scratch), g_sync_scratch);
        if (err != cudaSuccess) return int(err);
        g_scratch_addr[dev].store(scratch, std::memory_order_release);
    }
    // Every float the second phase reads is written by the first phase of the same call, so nothing left in the
    // array by an earlier call can leak into this one and nothing has to be cleared.
    SyncParams p = p_in;
    p.sum_out = scratch;
    p.sum_in = scratch;
    if (int rc = launch_sync_partial(p, shape, stream)) return rc;
    return launch_sync_finish(p, shape, stream);
}

}  // namespace qsr
