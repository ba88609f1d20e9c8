// Two-tier adapter store: every expert's adapters live in host memory, the experts in use are kept in a
// fixed number of HBM slots (the pools the LoRA kernels read), and a batch's missing experts are brought in
// with asynchronous host-to-device copies between the router and the forward pass.  Host code only: the
// kernels see nothing but the pools and the expert -> slot table they already read.
#include <vector>

#include "common.cuh"

struct moin_cache {
  int E = 0, n_slots = 0;
  std::vector<moin_cache_projection> projs;
  int32_t* dev_table = nullptr;        // [E] device: slot of every expert, -1 = not resident
  std::vector<int32_t> slot_of;        // host mirror of the table
  std::vector<int32_t> expert_in;      // [n_slots] expert held by a slot, -1 = free
  std::vector<uint64_t> last_used;     // [n_slots] tick of the last batch that used the slot
  uint64_t tick = 0;
  // pinned snapshots of the table for the asynchronous upload; an event guards the reuse of a snapshot
  static constexpr int kSnapshots = 4;
  int32_t* snap[kSnapshots] = {nullptr, nullptr, nullptr, nullptr};
  cudaEvent_t snap_done[kSnapshots] = {nullptr, nullptr, nullptr, nullptr};
  uint64_t uploads = 0;
};

using namespace moin;

extern "C" moin_status moin_cache_create(int32_t E, int32_t n_slots, const moin_cache_projection* projs,
                                         int32_t n_projs, int32_t* dev_slot_of_expert, moin_cache** out) {
  if (!out || E < 1 || n_slots < 1 || !projs || n_projs < 1 || !dev_slot_of_expert) return MOIN_ERR_INVALID_ARG;
  for (int p = 0; p < n_projs; ++p) {
    const moin_cache_projection& d = projs[p];
    if (!d.host_A || !d.host_B || !d.dev_A || !d.dev_B || d.r < 1 || d.d_in < 1 || d.d_out < 1) return MOIN_ERR_INVALID_ARG;
  }
  moin_cache* c = new moin_cache();
  c->E = E;
  c->n_slots = n_slots;
  c->projs.assign(projs, projs + n_projs);
  c->dev_table = dev_slot_of_expert;
  c->slot_of.assign(E, -1);
  c->expert_in.assign(n_slots, -1);
  c->last_used.assign(n_slots, 0);
  for (int i = 0; i < moin_cache::kSnapshots; ++i) {
    cudaError_t e = cudaHostAlloc((void**)&c->snap[i], sizeof(int32_t) * (size_t)E, cudaHostAllocDefault);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->snap_done[i], cudaEventDisableTiming);
    if (e != cudaSuccess) {
      moin_cache_destroy(c);
      return record_cuda(e);
    }
  }
  *out = c;
  return MOIN_OK;
}

extern "C" void moin_cache_destroy(moin_cache* c) {
  if (!c) return;
  for (int i = 0; i < moin_cache::kSnapshots; ++i) {
    if (c->snap_done[i]) {
      cudaEventSynchronize(c->snap_done[i]);
      cudaEventDestroy(c->snap_done[i]);
    }
    if (c->snap[i]) cudaFreeHost(c->snap[i]);
  }
  delete c;
}

extern "C" moin_status moin_cache_admit(moin_cache* c, const int32_t* expert_ids, int32_t n, moin_stream stream,
                                        int32_t* n_missed, uint64_t* bytes_copied) {
  if (!c || n < 0 || (n > 0 && !expert_ids)) return MOIN_ERR_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  c->tick += 1;
  // 1. distinct valid experts of the batch, in order of first appearance; hits are touched first so that no
  //    expert of this batch can be chosen as a victim
  std::vector<int32_t> wanted;
  std::vector<char> seen(c->E, 0);
  for (int i = 0; i < n; ++i) {
    const int32_t e = expert_ids[i];
    if (e < 0 || e >= c->E || seen[e]) continue;
    seen[e] = 1;
    wanted.push_back(e);
  }
  if ((int)wanted.size() > c->n_slots) return MOIN_ERR_WORKSPACE;   // the batch alone does not fit
  for (int32_t e : wanted)
    if (c->slot_of[e] >= 0) c->last_used[c->slot_of[e]] = c->tick;
  // 2. misses: free slot first, else the least recently used slot (lowest index on ties)
  int missed = 0;
  uint64_t bytes = 0;
  for (int32_t e : wanted) {
    if (c->slot_of[e] >= 0) continue;
    int victim = -1;
    for (int sl = 0; sl < c->n_slots; ++sl) {
      if (c->last_used[sl] == c->tick) continue;   // in use by this batch
      if (c->expert_in[sl] < 0) {
        victim = sl;
        break;
      }
      if (victim < 0 || c->last_used[sl] < c->last_used[victim]) victim = sl;
    }
    if (victim < 0) return MOIN_ERR_WORKSPACE;     // cannot happen: wanted.size() <= n_slots
    if (c->expert_in[victim] >= 0) c->slot_of[c->expert_in[victim]] = -1;
    c->expert_in[victim] = e;
    c->slot_of[e] = victim;
    c->last_used[victim] = c->tick;
    for (const moin_cache_projection& d : c->projs) {
      const size_t a_bytes = (size_t)d.r * (size_t)d.d_in * sizeof(__nv_bfloat16);
      const size_t b_bytes = (size_t)d.d_out * (size_t)d.r * sizeof(__nv_bfloat16);
      cudaError_t err = cudaMemcpyAsync((char*)d.dev_A + (size_t)victim * a_bytes, (const char*)d.host_A + (size_t)e * a_bytes,
                                        a_bytes, cudaMemcpyHostToDevice, s);
      if (err == cudaSuccess)
        err = cudaMemcpyAsync((char*)d.dev_B + (size_t)victim * b_bytes, (const char*)d.host_B + (size_t)e * b_bytes,
                              b_bytes, cudaMemcpyHostToDevice, s);
      if (err != cudaSuccess) return record_cuda(err);
      bytes += a_bytes + b_bytes;
    }
    ++missed;
  }
  // 3. the table the kernels read (uploaded on every call, so a fresh device table needs no initialisation)
  {
    const int i = (int)(c->uploads % moin_cache::kSnapshots);
    cudaError_t err = cudaEventSynchronize(c->snap_done[i]);   // the upload that last used this snapshot is done
    if (err != cudaSuccess) return record_cuda(err);
    for (int e = 0; e < c->E; ++e) c->snap[i][e] = c->slot_of[e];
    err = cudaMemcpyAsync(c->dev_table, c->snap[i], sizeof(int32_t) * (size_t)c->E, cudaMemcpyHostToDevice, s);
    if (err == cudaSuccess) err = cudaEventRecord(c->snap_done[i], s);
    if (err != cudaSuccess) return record_cuda(err);
    c->uploads += 1;
  }
  if (n_missed) *n_missed = missed;
  if (bytes_copied) *bytes_copied = bytes;
  return MOIN_OK;
}

extern "C" moin_status moin_cache_slot_of(const moin_cache* c, int32_t expert, int32_t* slot) {
  if (!c || !slot || expert < 0 || expert >= c->E) return MOIN_ERR_INVALID_ARG;
  *slot = c->slot_of[expert];
  return MOIN_OK;
}
