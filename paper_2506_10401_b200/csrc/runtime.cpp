#include "runtime.h"

#include <dlfcn.h>

#include <cstdlib>
#include <cstring>
#include <fstream>
#include <functional>
#include <map>
#include <mutex>
#include <sstream>

#include "../../include/hct.h"
#include "driver.h"
#include "graph.h"

namespace hct {

namespace {

// ---- NVRTC, opened at first use
typedef int nvrtcResult;
typedef struct _nvrtcProgram* nvrtcProgram;
struct Nvrtc {
  nvrtcResult (*CreateProgram)(nvrtcProgram*, const char*, const char*, int, const char* const*, const char* const*);
  nvrtcResult (*CompileProgram)(nvrtcProgram, int, const char* const*);
  nvrtcResult (*GetCUBINSize)(nvrtcProgram, size_t*);
  nvrtcResult (*GetCUBIN)(nvrtcProgram, char*);
  nvrtcResult (*GetProgramLogSize)(nvrtcProgram, size_t*);
  nvrtcResult (*GetProgramLog)(nvrtcProgram, char*);
  nvrtcResult (*DestroyProgram)(nvrtcProgram*);
  const char* (*GetErrorString)(nvrtcResult);
};

const Nvrtc& nvrtc() {
  static Nvrtc api;
  static std::once_flag once;
  static std::string err;
  std::call_once(once, [] {
    const char* names[] = {"libnvrtc.so.12", "/usr/local/cuda/lib64/libnvrtc.so.12", "libnvrtc.so"};
    void* h = nullptr;
    if (const char* p = std::getenv("HCT_NVRTC_PATH")) h = dlopen(p, RTLD_NOW | RTLD_LOCAL);
    for (auto n : names)
      if (!h) h = dlopen(n, RTLD_NOW | RTLD_LOCAL);
    if (!h) {
      err = "cannot open libnvrtc.so.12 (set HCT_NVRTC_PATH)";
      return;
    }
#define HCT_SYM(field, sym)                                  \
  *(void**)(&api.field) = dlsym(h, sym);                     \
  if (!api.field && err.empty()) err = std::string("missing NVRTC symbol ") + sym;
    HCT_SYM(CreateProgram, "nvrtcCreateProgram")
    HCT_SYM(CompileProgram, "nvrtcCompileProgram")
    HCT_SYM(GetCUBINSize, "nvrtcGetCUBINSize")
    HCT_SYM(GetCUBIN, "nvrtcGetCUBIN")
    HCT_SYM(GetProgramLogSize, "nvrtcGetProgramLogSize")
    HCT_SYM(GetProgramLog, "nvrtcGetProgramLog")
    HCT_SYM(DestroyProgram, "nvrtcDestroyProgram")
    HCT_SYM(GetErrorString, "nvrtcGetErrorString")
#undef HCT_SYM
  });
  if (!err.empty()) throw Error(HCT_ERR_COMPILE, err);
  return api;
}

std::mutex g_cache_mu;
std::map<std::string, std::vector<char>> g_cubins;

}  // namespace

const std::vector<char>& compile_cubin(const std::string& source, const std::string& name) {
  {
    std::lock_guard<std::mutex> lk(g_cache_mu);
    auto it = g_cubins.find(source);
    if (it != g_cubins.end()) return it->second;
  }
  const Nvrtc& rt = nvrtc();
  nvrtcProgram prog = nullptr;
  nvrtcResult r = rt.CreateProgram(&prog, source.c_str(), (name + ".cu").c_str(), 0, nullptr, nullptr);
  if (r != 0) throw Error(HCT_ERR_COMPILE, std::string("nvrtcCreateProgram: ") + rt.GetErrorString(r));
  const char* opts[] = {"--gpu-architecture=sm_100a", "--std=c++17", "-lineinfo", "-default-device"};
  r = rt.CompileProgram(prog, 4, opts);
  if (r != 0) {
    size_t n = 0;
    rt.GetProgramLogSize(prog, &n);
    std::string log(n, '\0');
    if (n) rt.GetProgramLog(prog, &log[0]);
    rt.DestroyProgram(&prog);
    if (const char* dump = std::getenv("HCT_DUMP_FAILED")) {
      std::ofstream f(dump);
      f << source;
    }
    throw Error(HCT_ERR_COMPILE, "compiling " + name + " failed: " + log.substr(0, 4000));
  }
  size_t sz = 0;
  rt.GetCUBINSize(prog, &sz);
  std::vector<char> bin(sz);
  rt.GetCUBIN(prog, bin.data());
  rt.DestroyProgram(&prog);
  std::lock_guard<std::mutex> lk(g_cache_mu);
  return g_cubins.emplace(source, std::move(bin)).first->second;
}

const Driver& driver() {
  static Driver d;
  static std::once_flag once;
  static std::string err;
  std::call_once(once, [] {
    void* h = dlopen("libcuda.so.1", RTLD_NOW | RTLD_GLOBAL);
    if (!h) {
      err = "cannot open libcuda.so.1: no CUDA driver on this machine";
      return;
    }
#define HCT_SYM(field, sym)                                  \
  *(void**)(&d.field) = dlsym(h, sym);                       \
  if (!d.field && err.empty()) err = std::string("missing driver symbol ") + sym;
    HCT_SYM(Init, "cuInit")
    HCT_SYM(GetErrorString, "cuGetErrorString")
    HCT_SYM(DeviceGet, "cuDeviceGet")
    HCT_SYM(DeviceGetAttribute, "cuDeviceGetAttribute")
    HCT_SYM(DevicePrimaryCtxRetain, "cuDevicePrimaryCtxRetain")
    HCT_SYM(DevicePrimaryCtxRelease, "cuDevicePrimaryCtxRelease_v2")
    HCT_SYM(CtxPushCurrent, "cuCtxPushCurrent_v2")
    HCT_SYM(CtxPopCurrent, "cuCtxPopCurrent_v2")
    HCT_SYM(ModuleLoadData, "cuModuleLoadData")
    HCT_SYM(ModuleUnload, "cuModuleUnload")
    HCT_SYM(ModuleGetFunction, "cuModuleGetFunction")
    HCT_SYM(FuncSetAttribute, "cuFuncSetAttribute")
    HCT_SYM(OccupancyMaxActiveBlocksPerMultiprocessor, "cuOccupancyMaxActiveBlocksPerMultiprocessor")
    HCT_SYM(LaunchKernel, "cuLaunchKernel")
    HCT_SYM(LaunchKernelEx, "cuLaunchKernelEx")
    HCT_SYM(MemAlloc, "cuMemAlloc_v2")
    HCT_SYM(MemFree, "cuMemFree_v2")
    HCT_SYM(MemcpyDtoH, "cuMemcpyDtoH_v2")
    HCT_SYM(MemsetD8, "cuMemsetD8_v2")
    HCT_SYM(MemsetD8Async, "cuMemsetD8Async")
    HCT_SYM(EventCreate, "cuEventCreate")
    HCT_SYM(EventRecord, "cuEventRecord")
    HCT_SYM(EventSynchronize, "cuEventSynchronize")
    HCT_SYM(EventElapsedTime, "cuEventElapsedTime")
    HCT_SYM(EventDestroy, "cuEventDestroy_v2")
    HCT_SYM(TensorMapEncodeTiled, "cuTensorMapEncodeTiled")
#undef HCT_SYM
    if (err.empty()) {
      int rc = d.Init(0);
      if (rc != 0) err = "cuInit failed with code " + std::to_string(rc);
    }
  });
  if (!err.empty()) throw Error(HCT_ERR_CUDA, err);
  return d;
}

}  // namespace hct
