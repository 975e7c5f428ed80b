// Kernel skeleton sources, embedded by the build step from csrc/kernels/*.cuh.
#include <cstring>

#include "../../include/hct.h"
#include "codegen.h"

namespace hct {
namespace {
struct Skeleton {
  const char* name;
  const char* text;
};
#include "skeletons.inc"
}  // namespace

const char* skeleton_source(const char* name) {
  for (const auto& s : kSkeletons)
    if (std::strcmp(s.name, name) == 0) return s.text;
  throw Error(HCT_ERR_COMPILE, std::string("unknown kernel skeleton ") + name);
}
}  // namespace hct
