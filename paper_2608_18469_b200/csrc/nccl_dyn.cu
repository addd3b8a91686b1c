#include "nccl_dyn.cuh"

#include <dlfcn.h>

#include <cstdlib>
#include <mutex>

namespace erase {
namespace {

std::once_flag g_once;
NcclApi g_api;
bool g_ok = false;
std::string g_why;

void load() {
  void* h = nullptr;
  std::string tried;
  if (const char* path = getenv("ERASE_NCCL_LIB")) {
    h = dlopen(path, RTLD_NOW | RTLD_LOCAL);
    if (!h) tried += std::string(path) + ": " + dlerror() + "; ";
  }
  if (!h) {
    h = dlopen("libnccl.so.2", RTLD_NOW | RTLD_LOCAL);
    if (!h) tried += std::string("libnccl.so.2: ") + dlerror();
  }
  if (!h) {
    g_why = "NCCL could not be loaded (" + tried + ")";
    return;
  }
  auto sym = [&](const char* name, void** out) {
    *out = dlsym(h, name);
    if (!*out) g_why += std::string(g_why.empty() ? "NCCL lacks " : ", ") + name;
  };
  sym("ncclGetUniqueId", (void**)&g_api.get_unique_id);
  sym("ncclCommInitRank", (void**)&g_api.comm_init_rank);
  sym("ncclCommDestroy", (void**)&g_api.comm_destroy);
  sym("ncclAllReduce", (void**)&g_api.all_reduce);
  sym("ncclGetVersion", (void**)&g_api.get_version);
  sym("ncclGetErrorString", (void**)&g_api.error_string);
  g_ok = g_why.empty();
}

}  // namespace

const NcclApi* nccl_api(std::string* why) {
  std::call_once(g_once, load);
  if (!g_ok && why) *why = g_why;
  return g_ok ? &g_api : nullptr;
}

}  // namespace erase
