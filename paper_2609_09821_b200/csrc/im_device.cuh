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
__device__ __forceinline__ float dot(Vec3 a, Vec3 b) { return a.x * b.x + a.y * b.y + a.z * b.z; }
__device__ __forceinline__ Vec3 cross(Vec3 a, Vec3 b)
{
    return {a.y * b.z - a.z * b.y, a.z * b.x - a.x * b.z, a.x * b.y - a.y * b.x};
}

__device__ __forceinline__ Quat qmul(Quat a, Quat b)
{
    return {a.w * b.w - a.x * b.x - a.y * b.y - a.z * b.z,
            a.w * b.x + a.x * b.w + a.y * b.z - a.z * b.y,
            a.w * b.y - a.x * b.z + a.y * b.w + a.z * b.x,
            a.w * b.z + a.x * b.y - a.y * b.x + a.z * b.w};
}
__device__ __forceinline__ Quat qconj(Quat a) { return {a.w, -a.x, -a.y, -a.z}; }

// R(q) v for a unit quaternion: v + w t + u x t with t = 2 u x v.
__device__ __forceinline__ Vec3 qrot(Quat q, Vec3 v)
{
    Vec3 u = {q.x, q.y, q.z};
    Vec3 t = 2.0f * cross(u, v);
    return v + q.w * t + cross(u, t);
}
__device__ __forceinline__ Vec3 qrot_inv(Quat q, Vec3 v) { return qrot(qconj(q), v); }

// First and third columns of the rotation matrix (the "tangent" and "normal"
// of the 6-float orientation encoding of the observation).
__device__ __forceinline__ Vec3 qcol_x(Quat q)
{
    return {1.0f - 2.0f * (q.y * q.y + q.z * q.z), 2.0f * (q.x * q.y + q.w * q.z), 2.0f * (q.x * q.z - q.w * q.y)};
}
__device__ __forceinline__ Vec3 qcol_z(Quat q)
{
    return {2.0f * (q.x * q.z + q.w * q.y), 2.0f * (q.y * q.z - q.w * q.x), 1.0f - 2.0f * (q.x * q.x + q.y * q.y)};
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
