// The few CUDA driver entry points the library uses, resolved from libcuda.so.1 at first use.
// Types are declared locally so that no CUDA header is needed to build the host code.
#pragma once
#include <cstddef>
#include <cstdint>

namespace hct {

typedef int CUresult_t;
typedef int CUdevice_t;
typedef struct CUctx_st* CUcontext_t;
typedef struct CUmod_st* CUmodule_t;
typedef struct CUfunc_st* CUfunction_t;
typedef struct CUstream_st* CUstream_t;
typedef struct CUevent_st* CUevent_t;
typedef unsigned long long CUdeviceptr_t;

struct alignas(64) TensorMap {
  uint64_t opaque[16];
};

enum {
  kAttrComputeCapabilityMajor = 75,
  kAttrComputeCapabilityMinor = 76,
  kAttrMultiprocessorCount = 16,
  kAttrMaxSharedMemoryPerBlockOptin = 97,
  kFuncAttrMaxDynamicSharedSizeBytes = 8,
};

// cuLaunchKernelEx configuration (layout of CUlaunchConfig / CUlaunchAttribute)
struct LaunchAttr {
  int id;
  char pad[4];
  union {
    char pad64[64];
    int programmatic_stream_serialization_allowed;
  } value;
};
struct LaunchConfig {
  unsigned gridX, gridY, gridZ, blockX, blockY, blockZ, sharedMemBytes;
  CUstream_t stream;
  LaunchAttr* attrs;
  unsigned numAttrs;
};
enum { kLaunchAttrProgrammaticStreamSerialization = 6 };

struct Driver {
  CUresult_t (*Init)(unsigned);
  CUresult_t (*GetErrorString)(CUresult_t, const char**);
  CUresult_t (*DeviceGet)(CUdevice_t*, int);
  CUresult_t (*DeviceGetAttribute)(int*, int, CUdevice_t);
  CUresult_t (*DevicePrimaryCtxRetain)(CUcontext_t*, CUdevice_t);
  CUresult_t (*DevicePrimaryCtxRelease)(CUdevice_t);
  CUresult_t (*CtxPushCurrent)(CUcontext_t);
  CUresult_t (*CtxPopCurrent)(CUcontext_t*);
  CUresult_t (*ModuleLoadData)(CUmodule_t*, const void*);
  CUresult_t (*ModuleUnload)(CUmodule_t);
  CUresult_t (*ModuleGetFunction)(CUfunction_t*, CUmodule_t, const char*);
  CUresult_t (*FuncSetAttribute)(CUfunction_t, int, int);
  CUresult_t (*OccupancyMaxActiveBlocksPerMultiprocessor)(int*, CUfunction_t, int, size_t);
  CUresult_t (*LaunchKernel)(CUfunction_t, unsigned, unsigned, unsigned, unsigned, unsigned, unsigned, unsigned, CUstream_t,
                             void**, void**);
  CUresult_t (*LaunchKernelEx)(const LaunchConfig*, CUfunction_t, void**, void**);
  CUresult_t (*MemAlloc)(CUdeviceptr_t*, size_t);
  CUresult_t (*MemFree)(CUdeviceptr_t);
  CUresult_t (*MemcpyDtoH)(void*, CUdeviceptr_t, size_t);
  CUresult_t (*MemsetD8)(CUdeviceptr_t, unsigned char, size_t);
  CUresult_t (*MemsetD8Async)(CUdeviceptr_t, unsigned char, size_t, CUstream_t);
  CUresult_t (*EventCreate)(CUevent_t*, unsigned);
  CUresult_t (*EventRecord)(CUevent_t, CUstream_t);
  CUresult_t (*EventSynchronize)(CUevent_t);
  CUresult_t (*EventElapsedTime)(float*, CUevent_t, CUevent_t);
  CUresult_t (*EventDestroy)(CUevent_t);
  // CUtensorMap*, dtype, rank, globalAddress, globalDim, globalStrides, boxDim, elementStrides, interleave, swizzle,
  // l2Promotion, oobFill
  CUresult_t (*TensorMapEncodeTiled)(TensorMap*, int, unsigned, void*, const uint64_t*, const uint64_t*, const uint32_t*,
                                     const uint32_t*, int, int, int, int);
};

}  // namespace hct
