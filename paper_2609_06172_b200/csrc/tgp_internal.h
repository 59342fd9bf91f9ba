// Internal structures shared by the host planner and the device engine.
#pragma once
#include <cstdint>
#include <string>
#include <vector>
#include <map>
#include <tuple>
#include <thread>
#include "tgp.h"

struct TgpPool { char *host_base; uint64_t bytes; uint32_t flags; char *dev_alias; bool locked_by_us; };

struct TgpTensor {
    uint32_t pool; uint64_t off, size; uint64_t site_hash, counter; int32_t layer; uint32_t kind, flags;
};

struct TgpOp {
    uint32_t step; uint64_t site; int32_t layer; uint32_t kind; uint64_t flops, hbm;
    uint32_t acc0, nacc;                 // slice of TgpTrace::acc
};

struct TgpStep { uint32_t kind, op0, nops; };

struct TgpCmd {
    uint32_t seq; uint8_t kind; uint32_t tensor; uint64_t bytes, pool_off, arena_off;
    int32_t wait_op, first_use, release_after;
};
enum { CMD_H2D = 0, CMD_ALLOC = 1, CMD_D2H = 2 };
enum { CLS_LINK = 0, CLS_HBM = 1, CLS_COMPUTE = 2 };

struct TgpPlan {
    bool valid = false;
    uint32_t first_step = 0, first_op = 0;   // > 0: a tail plan made at that step boundary; arrays below are still sized for the whole trace
    std::vector<uint8_t> cls, crit, zc;
    std::vector<uint64_t> score;
    std::vector<std::pair<uint32_t, uint64_t>> pins;
    std::vector<uint32_t> kept;          // pins that were resident when the plan began (a tail plan that keeps pins): never placed
    uint64_t ring_base = 0, ring_size = 0;
    std::vector<TgpCmd> cmds;
    std::vector<uint64_t> totals;        // 4 per step
    // resolved placement of every access, parallel to the trace's access array: arena offset, or
    // UINT64_MAX for a zero-copy access (read in place in the pool)
    std::vector<uint64_t> acc_where;
    std::vector<int32_t> op_last_place;  // per op: index of its last H2D/ALLOC command, or -1
    std::vector<uint8_t> op_is_wait_target;
};

struct TgpRole { uint32_t kind; int32_t layer, expert; uint32_t block, row0, rows, tensor; };

struct TgpEngine;   // device-side state (tgp_engine.cu)

struct tgp_ctx {
    tgp_machine mach{};
    std::vector<TgpPool> pools;
    std::vector<TgpTensor> tensors;
    std::vector<uint32_t> by_addr;                       // tensor ids sorted by (pool, off)
    bool by_addr_dirty = false;
    std::map<uint64_t, uint64_t> site_counter;
    // trace
    bool tracing = false, traced = false;
    std::vector<TgpOp> ops;
    std::vector<tgp_access> acc;
    std::vector<TgpStep> steps;
    // policy inputs
    uint64_t budget = 0, object_bytes = 20ull << 20;
    uint32_t variant = TGP_VAR_EXPLICIT_RING, bits = TGP_BIT_A | TGP_BIT_P | TGP_BIT_ZC | TGP_BIT_W;
    std::vector<uint64_t> measured_ns;                   // runtime monitor: kernel time per op in ns (0 = not measured), or empty
    TgpPlan plan;
    // re-plan of the remaining steps while the run is under way: built on a helper thread, swapped in at its boundary
    TgpPlan tail_plan, base_plan;                        // base_plan: the whole-run plan set aside while a tail plan is in use
    std::thread replan_thread;
    bool tail_ready = false;
    bool replan_keep = false;            // tail plans keep the resident pins of the plan in use (tgp_set_replan_keep)
    int tail_rc = 0;
    uint32_t tail_step = 0;
    std::string tail_err;
    // model
    bool bound = false;
    tgp_model_cfg cfg{};
    std::vector<TgpRole> roles;
    std::vector<int32_t> role_of_tensor;                 // tensor id -> index in roles, or -1
    std::vector<float> router_bias;
    std::map<std::tuple<uint32_t, int32_t, int32_t>, std::vector<uint32_t>> role_index;   // (kind, layer, expert) -> roles by block
    std::vector<uint32_t> run_counts;                    // MoE: tokens routed per (step, layer, expert) in the current run
    TgpEngine *eng = nullptr;
    void *arena = nullptr; uint64_t arena_bytes = 0;
    std::string err;
};

int tgp_fail(tgp_ctx *ctx, int code, const std::string &msg);
void tgp_engine_free(tgp_ctx *ctx);
