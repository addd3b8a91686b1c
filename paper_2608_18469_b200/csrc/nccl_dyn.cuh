// NCCL, bound at run time.  The library has no link-time dependency on NCCL: a process that never
// asks for data-parallel replicas never loads it.  The first call of nccl_api() opens the NCCL the
// process already has (the one a framework loaded under the same soname), else the one the loader
// finds as "libnccl.so.2", else the file ERASE_NCCL_LIB names.  Only NCCL's public C interface is used:
// the few declarations below restate it (opaque communicator, 128-byte id, result code 0 = success,
// float32 = 7, sum = 0, as NCCL 2.x defines them).
#pragma once
#include <cuda_runtime.h>

#include <cstddef>
#include <string>

namespace erase {

constexpr int NCCL_ID_BYTES = 128;
struct NcclId { char bytes[NCCL_ID_BYTES]; };
typedef struct ncclComm* NcclComm;

struct NcclApi {
  int (*get_unique_id)(NcclId*) = nullptr;
  int (*comm_init_rank)(NcclComm*, int nranks, NcclId id, int rank) = nullptr;
  int (*comm_destroy)(NcclComm) = nullptr;
  int (*all_reduce)(const void* send, void* recv, size_t count, int dtype, int op, NcclComm, cudaStream_t) = nullptr;
  int (*get_version)(int*) = nullptr;
  const char* (*error_string)(int) = nullptr;
};
constexpr int NCCL_FLOAT32 = 7;
constexpr int NCCL_SUM = 0;

// nullptr when no NCCL can be loaded; *why then says what was tried.  Thread-safe; the handle stays
// open for the life of the process.
const NcclApi* nccl_api(std::string* why);

}  // namespace erase
