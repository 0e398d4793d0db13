// The per-replica B operand of an MP-LoRA layer, in its two storage forms.
//
//   master copy (Algorithm 1):  one fp32 B per tensor; replica n uses B + k_n eps z_i, with z_i
//       regenerated from the Philox counter (never stored);
//   stored pair (Algorithm 2, "Mobile MP-LoRA", q = 1):  B[0] = B + eps z and B[1] = B - eps z are
//       kept in memory; replica n uses B[n & 1] as stored.
//
// Both forms are served as a (mean, signed perturbation) split, mean + pert = the replica's B.  The
// tensor-core form of the layer rounds the two parts to bf16 separately, so the perturbation keeps
// its resolution whatever the magnitude of B; the CUDA-core forms add them in fp32.
#pragma once
#include "common.cuh"
#include "kernels.h"

namespace zo {

// Elements e .. e+3 (e a multiple of 4) of slot `slot`, for replica `rep` of the step.
__device__ __forceinline__ void lora_operand(const LoraDesc& L, int slot, size_t e, int rep, float4& mean,
                                             float4& pert) {
  const size_t off = (size_t)slot * L.r * L.width + e;
  const float4 b0 = *reinterpret_cast<const float4*>(L.B + off);
  if (L.B1) {
    const float4 b1 = *reinterpret_cast<const float4*>(L.B1 + off);
    const float h = (rep & 1) ? -0.5f : 0.5f;
    mean = make_float4(0.5f * (b0.x + b1.x), 0.5f * (b0.y + b1.y), 0.5f * (b0.z + b1.z), 0.5f * (b0.w + b1.w));
    pert = make_float4(h * (b0.x - b1.x), h * (b0.y - b1.y), h * (b0.z - b1.z), h * (b0.w - b1.w));
    return;
  }
  mean = b0;
  pert = make_float4(0.f, 0.f, 0.f, 0.f);
  if (L.eps != 0.f) {
    const float s = (rep & 1) ? -L.eps : L.eps;
    const float4 z = z_block(L.seed, L.tensor_base + slot, (uint32_t)(rep >> 1), (uint32_t)(e >> 2));
    pert = make_float4(s * z.x, s * z.y, s * z.z, s * z.w);
  }
}

// The replica's B itself in fp32: B + k eps z (one fused multiply-add per element), or the stored B[n & 1].
__device__ __forceinline__ float4 lora_replica_b(const LoraDesc& L, int slot, size_t e, int rep) {
  const size_t off = (size_t)slot * L.r * L.width + e;
  if (L.B1) return *reinterpret_cast<const float4*>(((rep & 1) ? L.B1 : L.B) + off);
  float4 b = *reinterpret_cast<const float4*>(L.B + off);
  if (L.eps != 0.f) {
    const float s = (rep & 1) ? -L.eps : L.eps;
    const float4 z = z_block(L.seed, L.tensor_base + slot, (uint32_t)(rep >> 1), (uint32_t)(e >> 2));
    b.x = fmaf(s, z.x, b.x); b.y = fmaf(s, z.y, b.y); b.z = fmaf(s, z.z, b.z); b.w = fmaf(s, z.w, b.w);
  }
  return b;
}

}  // namespace zo
