// Tensor-core (tcgen05) dense transforms of the BF16 path -- placeholder interface: until the
// tcgen05 kernels land every shape reports "not supported" and the callers use the SIMT kernels.
#pragma once
#include "common.cuh"
#include "scan_sort.cuh"

struct TcState {
    int *err_word = nullptr;
};
static bool tc_init(TcState &, std::string &) { return true; }
static void tc_destroy(TcState &) {}
static lp_status tc_check(TcState &, Exec &, bool, std::string &) { return LP_OK; }
static bool tc_linear_supported(int, int) { return false; }
static bool tc_weight_grad_supported(int, int) { return false; }
static int64_t tc_weight_grad_partials(int64_t, int, int) { return 0; }
static bool tc_linear(TcState &, Exec &, int64_t, int, int, const bf16 *, int, const float *, bool, const float *, bool, bf16 *, int, std::string &e) { e = "not built"; return false; }
static bool tc_linear_bf16_b(TcState &, Exec &, int64_t, int, int, const bf16 *, int, const bf16 *, bool, const float *, bool, bf16 *, int, std::string &e) { e = "not built"; return false; }
static bool tc_weight_grad(TcState &, Exec &, int64_t, int, int, const bf16 *, int, const bf16 *, int, float *, int, float *, std::string &e) { e = "not built"; return false; }
