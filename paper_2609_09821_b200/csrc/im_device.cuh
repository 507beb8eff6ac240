// Device-side helpers shared by the kernels of the imitation-step library:
// quaternion algebra (w,x,y,z, Hamilton, R(q)v = q v q*), Philox4x32-10.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace im {

#define IM_STREAM_RESET 0u
#define IM_STREAM_ACTION 1u
#define IM_STREAM_RESET_NOISE 2u

struct Quat { float w, x, y, z; };
struct Vec3 { float x, y, z; };

__device__ __forceinline__ Vec3 operator+(Vec3 a, Vec3 b) { return {a.x + b.x, a.y + b.y, a.z + b.z}; }
__device__ __forceinline__ Vec3 operator-(Vec3 a, Vec3 b) { return {a.x - b.x, a.y - b.y, a.z - b.z}; }
__device__ __forceinline__ Vec3 operator*(float s, Vec3 a) { return {s * a.x, s * a.y, s * a.z}; }
__device__ __forceinline__ float dot(Vec3 a, Vec3 b) { return fmaf(a.z, b.z, fmaf(a.y, b.y, a.x * b.x)); }
__device__ __forceinline__ Vec3 cross(Vec3 a, Vec3 b)
{
    return {fmaf(a.y, b.z, -(a.z * b.y)), fmaf(a.z, b.x, -(a.x * b.z)), fmaf(a.x, b.y, -(a.y * b.x))};
}
// c + a x b
__device__ __forceinline__ Vec3 cross_add(Vec3 a, Vec3 b, Vec3 c)
{
    return {fmaf(a.y, b.z, fmaf(-a.z, b.y, c.x)), fmaf(a.z, b.x, fmaf(-a.x, b.z, c.y)), fmaf(a.x, b.y, fmaf(-a.y, b.x, c.z))};
}

__device__ __forceinline__ Quat qmul(Quat a, Quat b)
{
    return {fmaf(-a.z, b.z, fmaf(-a.y, b.y, fmaf(-a.x, b.x, a.w * b.w))),
            fmaf(-a.z, b.y, fmaf(a.y, b.z, fmaf(a.x, b.w, a.w * b.x))),
            fmaf(a.z, b.x, fmaf(a.y, b.w, fmaf(-a.x, b.z, a.w * b.y))),
            fmaf(a.z, b.w, fmaf(-a.y, b.x, fmaf(a.x, b.y, a.w * b.z)))};
}
__device__ __forceinline__ Quat qconj(Quat a) { return {a.w, -a.x, -a.y, -a.z}; }
// a* b
__device__ __forceinline__ Quat qmul_conj(Quat a, Quat b) { return qmul(qconj(a), b); }

// add + R(q) v for a unit quaternion: v + 2 w (u x v) + 2 u x (u x v).
__device__ __forceinline__ Vec3 qrot_add(Quat q, Vec3 v, Vec3 add)
{
    const Vec3 u = {q.x, q.y, q.z};
    const Vec3 t = cross(u, v);
    const Vec3 u2 = {u.x + u.x, u.y + u.y, u.z + u.z};
    const float w2 = q.w + q.w;
    const Vec3 base = {fmaf(w2, t.x, v.x + add.x), fmaf(w2, t.y, v.y + add.y), fmaf(w2, t.z, v.z + add.z)};
    return cross_add(u2, t, base);
}
__device__ __forceinline__ Vec3 qrot(Quat q, Vec3 v)
{
    const Vec3 u = {q.x, q.y, q.z};
    const Vec3 t = cross(u, v);
    const Vec3 u2 = {u.x + u.x, u.y + u.y, u.z + u.z};
    const float w2 = q.w + q.w;
    const Vec3 base = {fmaf(w2, t.x, v.x), fmaf(w2, t.y, v.y), fmaf(w2, t.z, v.z)};
    return cross_add(u2, t, base);
}
__device__ __forceinline__ Vec3 qrot_inv(Quat q, Vec3 v) { return qrot(qconj(q), v); }

// First and third columns of the rotation matrix (the "tangent" and "normal"
// of the 6-float orientation encoding of the observation).
__device__ __forceinline__ Vec3 qcol_x(Quat q)
{
    const float y2 = q.y + q.y, z2 = q.z + q.z;
    return {fmaf(-z2, q.z, fmaf(-y2, q.y, 1.0f)), fmaf(y2, q.x, z2 * q.w), fmaf(z2, q.x, -(y2 * q.w))};
}
__device__ __forceinline__ Vec3 qcol_z(Quat q)
{
    const float x2 = q.x + q.x, y2 = q.y + q.y;
    return {fmaf(x2, q.z, y2 * q.w), fmaf(y2, q.z, -(x2 * q.w)), fmaf(-y2, q.y, fmaf(-x2, q.x, 1.0f))};
}

// Rotation angle in [0, pi] of the rotation taking frame a to frame b.
__device__ __forceinline__ float rel_angle(Quat a, Quat b)
{
    Quat r = qmul(qconj(a), b);
    float n = sqrtf(r.x * r.x + r.y * r.y + r.z * r.z);
    return 2.0f * atan2f(n, fabsf(r.w));
}

__device__ __forceinline__ uint4 philox4x32_10(uint4 c, uint2 k)
{
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        if (r > 0) { k.x += 0x9E3779B9u; k.y += 0xBB67AE85u; }
        const uint32_t hi0 = __umulhi(0xD2511F53u, c.x), lo0 = 0xD2511F53u * c.x;
        const uint32_t hi1 = __umulhi(0xCD9E8D57u, c.z), lo1 = 0xCD9E8D57u * c.z;
        c = make_uint4(hi1 ^ c.y ^ k.x, lo1, hi0 ^ c.w ^ k.y, lo0);
    }
    return c;
}

// Two standard normals from two Philox words (Box-Muller): u1 in (0,1], u2 in [0,1).
__device__ __forceinline__ void box_muller(uint32_t x0, uint32_t x1, float &z0, float &z1)
{
    const float u1 = (float)((x0 >> 8) + 1u) * 5.9604644775390625e-08f;
    const float u2 = (float)(x1 >> 8) * 5.9604644775390625e-08f;
    // fast intrinsics: absolute error below 1e-6 on z, far inside the 1e-4 the sampled noise needs
    const float rad = sqrtf(-2.0f * __logf(u1));
    float s, c;
    __sincosf(6.283185307179586f * u2, &s, &c);
    z0 = rad * c;
    z1 = rad * s;
}

}  // namespace im
