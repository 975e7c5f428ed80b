// Run-time compilation (NVRTC) and the thin layer over the CUDA driver API.
// Both libraries are opened lazily so that the library itself loads, and graphs can be planned
// and compiled, on a machine without a GPU driver.
#pragma once
#include <string>
#include <vector>

namespace hct {

// Compile one translation unit to an sm_100a cubin.  Results are cached per process by source text.
// Throws Error(HCT_ERR_COMPILE) with the compiler log on failure.
const std::vector<char>& compile_cubin(const std::string& source, const std::string& name);

struct Driver;  // table of driver entry points
// Loads libcuda on first use; throws Error(HCT_ERR_CUDA) if it is missing.
const Driver& driver();

}  // namespace hct
