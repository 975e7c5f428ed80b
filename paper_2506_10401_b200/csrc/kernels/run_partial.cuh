// Runs of up to 32 consecutive epilogue elements whose first address is aligned to VW elements only
// (VW = 2 or 4 for bf16, 2 for fp32; included after tc_common.cuh): whole groups of VW elements move in
// one access, a ragged last group element by element.  Used where a tile's rows are not whole 16-byte
// vectors (images 28, 14 or 12 pixels wide), which would otherwise fall back to one access per element.
template <int VW>
__device__ __forceinline__ void hct_ld_run32w(const hct_bf16_t* p, float* v, int n) {
#pragma unroll
  for (int g = 0; g < 32 / VW; ++g) {
    if ((g + 1) * VW <= n) {
      if (VW == 4) {
        const uint2 t = __ldg((const uint2*)p + g);
        v[4 * g] = __uint_as_float(t.x << 16); v[4 * g + 1] = __uint_as_float(t.x & 0xffff0000u);
        v[4 * g + 2] = __uint_as_float(t.y << 16); v[4 * g + 3] = __uint_as_float(t.y & 0xffff0000u);
      } else {
        const unsigned t = __ldg((const unsigned*)p + g);
        v[2 * g] = __uint_as_float(t << 16); v[2 * g + 1] = __uint_as_float(t & 0xffff0000u);
      }
    } else {
#pragma unroll
      for (int j = 0; j < VW; ++j) v[g * VW + j] = g * VW + j < n ? hct_bf16_to_f32(__ldg(p + g * VW + j)) : 0.0f;
    }
  }
}
template <int VW>
__device__ __forceinline__ void hct_ld_run32w(const float* p, float* v, int n) {
#pragma unroll
  for (int g = 0; g < 16; ++g) {
    if ((g + 1) * 2 <= n) {
      const float2 t = __ldg((const float2*)p + g);
      v[2 * g] = t.x; v[2 * g + 1] = t.y;
    } else {
#pragma unroll
      for (int j = 0; j < 2; ++j) v[g * 2 + j] = g * 2 + j < n ? __ldg(p + g * 2 + j) : 0.0f;
    }
  }
}
template <int VW>
__device__ __forceinline__ void hct_st_run32w(hct_bf16_t* p, const float* v, int n) {
#pragma unroll
  for (int g = 0; g < 32 / VW; ++g) {
    if ((g + 1) * VW <= n) {
      if (VW == 4)
        ((uint2*)p)[g] = make_uint2(hct_pack_bf16x2(v[4 * g], v[4 * g + 1]), hct_pack_bf16x2(v[4 * g + 2], v[4 * g + 3]));
      else
        ((unsigned*)p)[g] = hct_pack_bf16x2(v[2 * g], v[2 * g + 1]);
    } else {
#pragma unroll
      for (int j = 0; j < VW; ++j)
        if (g * VW + j < n) p[g * VW + j] = hct_f32_to_bf16(v[g * VW + j]);
    }
  }
}
template <int VW>
__device__ __forceinline__ void hct_st_run32w(float* p, const float* v, int n) {
#pragma unroll
  for (int g = 0; g < 16; ++g) {
    if ((g + 1) * 2 <= n) {
      ((float2*)p)[g] = make_float2(v[2 * g], v[2 * g + 1]);
    } else {
#pragma unroll
      for (int j = 0; j < 2; ++j)
        if (g * 2 + j < n) p[g * 2 + j] = v[g * 2 + j];
    }
  }
}
