// A second memory tier under the slice cache (Section 5: all weights live in a large, slow store and are brought
// into the fast memory only when a slice misses).  Here the fast memory is a pool of slots in device memory, the
// slow store pinned host memory, and a miss is a copy of the slice's record on a side stream.  The cache decisions
// are the host bookkeeping of slicemoe_dbsc_*; this file keeps the bytes where the decisions say they are, and the
// device expert tables pointing at them.
//
// A record is what one slice of one expert consists of, back to back:
//   MSB record: gate MSB plane, gate scales, gate zero-points, then the same of up, then of down
//   LSB record: gate LSB plane, up LSB plane, down LSB plane
// and the store holds, for (layer l, expert e), the MSB record followed by the LSB record at
// (l * n_experts + e) * (msb_record + lsb_record).
// In the store a plane of a slice narrower than four bits (MAT63, MAT42) is kept dense - the bit stream of
// slicemoe_compact_plane - so a miss moves 3 or 2 bits per weight, not 4; the copy then lands in a staging buffer
// and one small kernel on the side stream spreads it into the slot's nibble planes.
// Every slot of the pool has the size of the larger record in its device form (rounded up to 256 bytes), so any slice fits any slot;
// slot 0 is never given out: table entries of slices that are not resident point there, so that a list naming
// an expert the caller did not request reads defined bytes, never an address outside the pool.
#include <algorithm>
#include <new>
#include <unordered_map>
#include <vector>

#include "common.cuh"

namespace {

inline uint64_t tier_key(int layer, int expert) {
  return (static_cast<uint64_t>(static_cast<uint32_t>(layer)) << 32) | static_cast<uint32_t>(expert);
}
inline size_t round256(size_t v) { return (v + 255) & ~static_cast<size_t>(255); }

struct MatBytes {
  size_t plane, scale, zp;  // plane: in the device (nibble) form
};

// One record from its stored form (in `src`, device staging) to its device form (in a slot): up to three planes as
// dense bit streams of `bits` bits per value -> nibble planes, and whatever follows each plane copied as it is.
struct ExpandJob {
  unsigned long long src_plane[3], dst_plane[3], words[3];  // byte offsets; 32-bit plane words
  unsigned long long src_meta[3], dst_meta[3], meta_bytes[3];
  int bits;
};
__global__ void tier_expand_kernel(const uint8_t* __restrict__ src, uint8_t* __restrict__ dst, ExpandJob job) {
  const size_t stride = (size_t)gridDim.x * blockDim.x, tid = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  const uint32_t mask = (1u << job.bits) - 1u;
  for (int m = 0; m < 3; ++m) {
    const uint8_t* in = src + job.src_plane[m];
    uint32_t* out = reinterpret_cast<uint32_t*>(dst + job.dst_plane[m]);
    for (size_t i = tid; i < job.words[m]; i += stride) {
      uint32_t packed = 0;
      for (int b = 0; b < job.bits; ++b) packed |= (uint32_t)in[i * job.bits + b] << (8 * b);
      uint32_t w = 0;
#pragma unroll
      for (int j = 0; j < 8; ++j) w |= ((packed >> (job.bits * j)) & mask) << (4 * j);
      out[i] = w;
    }
    for (size_t i = tid; i < job.meta_bytes[m]; i += stride) dst[job.dst_meta[m] + i] = src[job.src_meta[m] + i];
  }
}
inline MatBytes mat_bytes(int N, int K, int group) {
  const size_t w = static_cast<size_t>(N) * static_cast<size_t>(K);
  return MatBytes{w / 2, w / static_cast<size_t>(group) * 2, w / static_cast<size_t>(group)};
}

}  // namespace

namespace {
inline int stored_bits(int width) { return width < 4 ? width : 4; }
inline size_t stored_plane(size_t plane_bytes, int bits) { return plane_bytes / 4 * bits; }  // plane_bytes = N*K/2
}  // namespace

struct slicemoe_tier {
  slicemoe_shape shape;
  int n_layers;
  MatBytes gu, dn;           // gate/up [inter, hidden] and down [hidden, inter]
  size_t msb_rec, lsb_rec, slot_bytes;  // records in their device form
  int msb_bits, lsb_bits;               // stored bits per slice value (4: stored as on the device)
  size_t msb_rec_st, lsb_rec_st;        // records as stored
  uint8_t* staging;                     // device; only for stored forms that differ
  const uint8_t* store;      // pinned host
  uint8_t* pool;             // device
  int n_slots;
  slicemoe_expert* tables_dev;             // device [n_layers * n_experts]
  std::vector<slicemoe_expert> tables;     // host mirror
  std::vector<int> free_slots;
  std::unordered_map<uint64_t, int> msb_slot, lsb_slot;
  // Slices of the list being served that the cache no longer counts (a later entry of the same list pushed them
  // out, or they never fitted): their bytes stay where they are until the next request, because the launch that
  // follows this request reads them.  2 * top_k slots of the pool are set aside for them.
  std::vector<std::pair<uint64_t, int>> transient;  // (key, 1 = LSB slice)
  slicemoe_dbsc* cache;
  cudaEvent_t ev_compute, ev_copy;
  int64_t bytes_copied, copies;

  void point_msb(slicemoe_expert& ex, const uint8_t* rec) const {
    slicemoe_mat* m[3] = {&ex.gate, &ex.up, &ex.down};
    for (int i = 0; i < 3; ++i) {
      const MatBytes& b = i < 2 ? gu : dn;
      m[i]->msb = rec;
      m[i]->scale = reinterpret_cast<const uint16_t*>(rec + b.plane);
      m[i]->zp = rec + b.plane + b.scale;
      rec += b.plane + b.scale + b.zp;
    }
  }
  // Brings one record (part 0: MSB, 1: LSB) of store entry `idx` into the slot at `dst`, on stream `xs`.
  int fetch(size_t idx, int part, uint8_t* dst, cudaStream_t xs) {
    const size_t rec_st = msb_rec_st + lsb_rec_st;
    const uint8_t* src = store + idx * rec_st + (part ? msb_rec_st : 0);
    const size_t bytes = part ? lsb_rec_st : msb_rec_st;
    const int bits = part ? lsb_bits : msb_bits;
    if (bits == 4) {  // stored as on the device
      SM_CUDA_TRY(cudaMemcpyAsync(dst, src, bytes, cudaMemcpyHostToDevice, xs));
    } else {
      // the staging buffer is free again: whatever used it last ran earlier on this same stream
      SM_CUDA_TRY(cudaMemcpyAsync(staging, src, bytes, cudaMemcpyHostToDevice, xs));
      ExpandJob job;
      job.bits = bits;
      unsigned long long so = 0, d_o = 0;
      for (int i = 0; i < 3; ++i) {
        const MatBytes& b = i < 2 ? gu : dn;
        job.src_plane[i] = so;
        job.dst_plane[i] = d_o;
        job.words[i] = b.plane / 4;
        so += stored_plane(b.plane, bits);
        d_o += b.plane;
        job.src_meta[i] = so;
        job.dst_meta[i] = d_o;
        job.meta_bytes[i] = part ? 0 : b.scale + b.zp;
        so += job.meta_bytes[i];
        d_o += job.meta_bytes[i];
      }
      tier_expand_kernel<<<64, 256, 0, xs>>>(staging, dst, job);
      SM_LAUNCH_CHECK();
    }
    bytes_copied += static_cast<int64_t>(bytes);
    ++copies;
    return SLICEMOE_OK;
  }
  void point_lsb(slicemoe_expert& ex, const uint8_t* rec, bool resident) const {
    slicemoe_mat* m[3] = {&ex.gate, &ex.up, &ex.down};
    for (int i = 0; i < 3; ++i) {
      m[i]->lsb = resident ? rec : nullptr;  // a missing LSB plane is NULL: the kernels report it instead of reading it
      rec += (i < 2 ? gu : dn).plane;
    }
  }
};


extern "C" int slicemoe_tier_sizes(const slicemoe_shape* s, size_t* msb_record, size_t* lsb_record, size_t* slot_bytes,
                                   size_t* staging_bytes) {
  if (!s || s->hidden <= 0 || s->inter <= 0 || (s->hidden % 128) || (s->inter % 128) || !slicemoe::valid_group(s->group))
    return SLICEMOE_E_INVALID_ARG;
  if (!slicemoe::valid_widths(s->b_high, s->b_low)) return SLICEMOE_E_UNSUPPORTED;
  const MatBytes gu = mat_bytes(s->inter, s->hidden, s->group), dn = mat_bytes(s->hidden, s->inter, s->group);
  const int mb = stored_bits(s->b_low), lb = stored_bits(s->b_high - s->b_low);
  const size_t m = 2 * (gu.plane + gu.scale + gu.zp) + dn.plane + dn.scale + dn.zp, l = 2 * gu.plane + dn.plane;
  const size_t ms = 2 * (stored_plane(gu.plane, mb) + gu.scale + gu.zp) + stored_plane(dn.plane, mb) + dn.scale + dn.zp;
  const size_t ls = 2 * stored_plane(gu.plane, lb) + stored_plane(dn.plane, lb);
  if (msb_record) *msb_record = ms;
  if (lsb_record) *lsb_record = ls;
  if (slot_bytes) *slot_bytes = round256(std::max(m, l));
  if (staging_bytes) *staging_bytes = (mb < 4 || lb < 4) ? round256(std::max(ms, ls)) : 0;
  return SLICEMOE_OK;
}

extern "C" int slicemoe_tier_store_expert(const slicemoe_shape* s, const slicemoe_expert* expert, void* record_host,
                                          void* scratch_device, void* stream) {
  if (!s || !expert || !record_host) return SLICEMOE_E_INVALID_ARG;
  size_t ms = 0, ls = 0, stg = 0;
  const int rc = slicemoe_tier_sizes(s, &ms, &ls, nullptr, &stg);
  if (rc != SLICEMOE_OK) return rc;
  if (stg != 0 && !scratch_device) return SLICEMOE_E_INVALID_ARG;
  const MatBytes gu = mat_bytes(s->inter, s->hidden, s->group), dn = mat_bytes(s->hidden, s->inter, s->group);
  const int bits[2] = {stored_bits(s->b_low), stored_bits(s->b_high - s->b_low)};
  const slicemoe_mat* mats[3] = {&expert->gate, &expert->up, &expert->down};
  uint8_t* p = static_cast<uint8_t*>(record_host);
  cudaStream_t st = (cudaStream_t)stream;
  for (int part = 0; part < 2; ++part) {
    for (int i = 0; i < 3; ++i) {
      const MatBytes& b = i < 2 ? gu : dn;
      const void* plane = part ? mats[i]->lsb : mats[i]->msb;
      if (!plane || !mats[i]->scale || !mats[i]->zp) return SLICEMOE_E_INVALID_ARG;
      const size_t sp = stored_plane(b.plane, bits[part]);
      if (bits[part] < 4) {  // dense form first, in the scratch (the copies and kernels of one stream run in order)
        const int r2 = slicemoe_compact_plane(plane, mats[i]->N, mats[i]->K, bits[part], scratch_device, stream);
        if (r2 != SLICEMOE_OK) return r2;
        SM_CUDA_TRY(cudaMemcpyAsync(p, scratch_device, sp, cudaMemcpyDeviceToHost, st));
      } else {
        SM_CUDA_TRY(cudaMemcpyAsync(p, plane, sp, cudaMemcpyDeviceToHost, st));
      }
      p += sp;
      if (part == 0) {
        SM_CUDA_TRY(cudaMemcpyAsync(p, mats[i]->scale, b.scale, cudaMemcpyDeviceToHost, st));
        SM_CUDA_TRY(cudaMemcpyAsync(p + b.scale, mats[i]->zp, b.zp, cudaMemcpyDeviceToHost, st));
        p += b.scale + b.zp;
      }
    }
  }
  return SLICEMOE_OK;
}

extern "C" slicemoe_tier* slicemoe_tier_create(const slicemoe_shape* s, int n_layers, const void* store_host,
                                               void* pool_device, size_t pool_bytes, slicemoe_expert* tables_device,
                                               void* staging_device, size_t staging_bytes, double miss_budget,
                                               int warmup_steps, void* stream) {
  if (!s || n_layers <= 0 || !store_host || !pool_device || !tables_device || s->n_experts <= 0) return nullptr;
  if (reinterpret_cast<uintptr_t>(pool_device) & 255) return nullptr;
  size_t ms = 0, ls = 0, slot = 0, stg = 0;
  if (slicemoe_tier_sizes(s, &ms, &ls, &slot, &stg) != SLICEMOE_OK) return nullptr;
  if (stg != 0 && (!staging_device || staging_bytes < stg || (reinterpret_cast<uintptr_t>(staging_device) & 15))) return nullptr;
  const long long n_slots = static_cast<long long>(pool_bytes / slot);
  // slot 0 is the stand-in, 2 * top_k slots are set aside for slices in transit (see `transient`), the cache
  // gets the rest and must be able to hold one request list
  if (n_slots < 1 + 4LL * s->top_k || n_slots > (1 << 30)) return nullptr;
  slicemoe_tier* t = new (std::nothrow) slicemoe_tier();
  if (!t) return nullptr;
  t->shape = *s;
  t->n_layers = n_layers;
  t->gu = mat_bytes(s->inter, s->hidden, s->group);
  t->dn = mat_bytes(s->hidden, s->inter, s->group);
  t->msb_rec = 2 * (t->gu.plane + t->gu.scale + t->gu.zp) + t->dn.plane + t->dn.scale + t->dn.zp;
  t->lsb_rec = 2 * t->gu.plane + t->dn.plane;
  t->msb_bits = stored_bits(s->b_low);
  t->lsb_bits = stored_bits(s->b_high - s->b_low);
  t->msb_rec_st = ms;
  t->lsb_rec_st = ls;
  t->staging = static_cast<uint8_t*>(staging_device);
  t->slot_bytes = slot;
  t->store = static_cast<const uint8_t*>(store_host);
  t->pool = static_cast<uint8_t*>(pool_device);
  t->n_slots = static_cast<int>(n_slots);
  t->tables_dev = tables_device;
  t->bytes_copied = t->copies = 0;
  t->ev_compute = t->ev_copy = nullptr;
  // the cache counts slots: both slice kinds are charged one slot's bytes, which is what they occupy here
  t->cache = slicemoe_dbsc_create(static_cast<int64_t>(n_slots - 1 - 2 * s->top_k) * static_cast<int64_t>(slot), static_cast<int64_t>(slot),
                                  static_cast<int64_t>(slot), miss_budget, warmup_steps);
  bool ok = t->cache != nullptr && slicemoe_dbsc_log_evictions(t->cache, 1) == SLICEMOE_OK;
  ok = ok && cudaEventCreateWithFlags(&t->ev_compute, cudaEventDisableTiming) == cudaSuccess;
  ok = ok && cudaEventCreateWithFlags(&t->ev_copy, cudaEventDisableTiming) == cudaSuccess;
  if (ok) {
    try {
      for (int i = t->n_slots - 1; i >= 1; --i) t->free_slots.push_back(i);
      slicemoe_expert blank;
      slicemoe_mat* mm[3] = {&blank.gate, &blank.up, &blank.down};
      for (int i = 0; i < 3; ++i) {
        mm[i]->N = i < 2 ? s->inter : s->hidden;
        mm[i]->K = i < 2 ? s->hidden : s->inter;
      }
      t->point_msb(blank, t->pool);
      t->point_lsb(blank, t->pool, false);
      t->tables.assign(static_cast<size_t>(n_layers) * s->n_experts, blank);
    } catch (...) {
      ok = false;
    }
  }
  cudaStream_t st = (cudaStream_t)stream;
  ok = ok && cudaMemsetAsync(t->pool, 0, slot, st) == cudaSuccess;
  ok = ok && cudaMemcpyAsync(tables_device, t->tables.data(), t->tables.size() * sizeof(slicemoe_expert),
                             cudaMemcpyHostToDevice, st) == cudaSuccess;
  ok = ok && cudaStreamSynchronize(st) == cudaSuccess;  // the mirror is pageable: the copy has left it before we return
  if (!ok) {
    (void)cudaGetLastError();
    if (t->ev_compute) cudaEventDestroy(t->ev_compute);
    if (t->ev_copy) cudaEventDestroy(t->ev_copy);
    if (t->cache) slicemoe_dbsc_destroy(t->cache);
    delete t;
    return nullptr;
  }
  return t;
}

extern "C" void slicemoe_tier_destroy(slicemoe_tier* t) {
  if (!t) return;
  cudaEventDestroy(t->ev_compute);
  cudaEventDestroy(t->ev_copy);
  slicemoe_dbsc_destroy(t->cache);
  delete t;
}

extern "C" slicemoe_dbsc* slicemoe_tier_cache(slicemoe_tier* t) { return t ? t->cache : nullptr; }

extern "C" int slicemoe_tier_request(slicemoe_tier* t, int step, int layer, const int32_t* ids, const uint8_t* prec_req,
                                     int n, uint8_t* prec_out, void* compute_stream, void* copy_stream) {
  if (!t || !ids || !prec_req || !prec_out || n < 0 || n > SLICEMOE_MAX_TOP_K || step < 0) return SLICEMOE_E_INVALID_ARG;
  if (layer < 0 || layer >= t->n_layers) return SLICEMOE_E_INVALID_ARG;
  for (int i = 0; i < n; ++i)
    if (ids[i] < 0 || ids[i] >= t->shape.n_experts) return SLICEMOE_E_INVALID_ARG;
  cudaStream_t cs = (cudaStream_t)compute_stream, xs = (cudaStream_t)copy_stream;
  try {
    // Nothing that is still being read may be overwritten: the copies start when the work already enqueued on
    // the compute stream has finished.  (A slice's bytes are needed by the very next launch, whose routing
    // depended on the launch before: there is nothing of this token to overlap them with.)
    SM_CUDA_TRY(cudaEventRecord(t->ev_compute, cs));
    SM_CUDA_TRY(cudaStreamWaitEvent(xs, t->ev_compute, 0));
    std::vector<size_t> dirty;  // table entries to send
    auto drop = [&](uint64_t k, int is_lsb) {  // the slice's slot is free again, its table entry points at the stand-in
      auto& map = is_lsb ? t->lsb_slot : t->msb_slot;
      auto it = map.find(k);
      if (it == map.end()) return;
      t->free_slots.push_back(it->second);
      map.erase(it);
      const size_t idx = static_cast<size_t>(k >> 32) * t->shape.n_experts + static_cast<size_t>(k & 0xffffffffu);
      if (is_lsb) t->point_lsb(t->tables[idx], t->pool, false);
      else t->point_msb(t->tables[idx], t->pool);
      dirty.push_back(idx);
    };
    // what the previous request kept beyond the cache's books has been read by now
    for (auto& tr : t->transient) drop(tr.first, tr.second);
    t->transient.clear();
    auto in_list = [&](uint64_t k) {
      for (int i = 0; i < n; ++i)
        if (tier_key(layer, ids[i]) == k) return true;
      return false;
    };
    auto release = [&]() -> int {
      int32_t el[64], ee[64];
      uint8_t il[64];
      for (;;) {
        const int m = slicemoe_dbsc_drain_evicted(t->cache, el, ee, il, 64);
        if (m < 0) return m;
        for (int i = 0; i < m; ++i) {
          const uint64_t k = tier_key(el[i], ee[i]);
          if (in_list(k)) t->transient.emplace_back(k, (int)il[i]);  // still needed by the coming launch
          else drop(k, il[i]);
        }
        if (m < 64) return SLICEMOE_OK;
      }
    };
    for (int i = 0; i < n; ++i) {
      int mh = 0, lh = 0;
      const int prec = slicemoe_dbsc_request(t->cache, step, layer, ids[i], prec_req[i] != 0, &mh, &lh, nullptr);
      if (prec < 0) return prec;
      prec_out[i] = static_cast<uint8_t>(prec);
      int rc = release();
      if (rc != SLICEMOE_OK) return rc;
      const uint64_t k = tier_key(layer, ids[i]);
      const size_t idx = static_cast<size_t>(layer) * t->shape.n_experts + ids[i];
      int has_m = 0, has_l = 0;
      slicemoe_dbsc_contains(t->cache, layer, ids[i], &has_m, &has_l);
      for (int part = 0; part < 2; ++part) {  // 0: MSB record (always needed), 1: LSB record (when run at both slices)
        if (part == 1 && !prec) continue;
        auto& map = part ? t->lsb_slot : t->msb_slot;
        const bool counted = (part ? has_l : has_m) != 0;
        auto tr = std::find(t->transient.begin(), t->transient.end(), std::make_pair(k, part));
        if (map.find(k) != map.end()) {  // the bytes are there
          if (counted && tr != t->transient.end()) t->transient.erase(tr);  // (the same expert twice in the list)
          continue;
        }
        if (t->free_slots.empty()) return SLICEMOE_E_UNSUPPORTED;  // cannot happen with the slots set aside
        const int slot = t->free_slots.back();
        t->free_slots.pop_back();
        map[k] = slot;
        if (!counted && tr == t->transient.end()) t->transient.emplace_back(k, part);  // used by this launch, not kept
        uint8_t* dst = t->pool + static_cast<size_t>(slot) * t->slot_bytes;
        rc = t->fetch(idx, part, dst, xs);
        if (rc != SLICEMOE_OK) return rc;
        if (part) t->point_lsb(t->tables[idx], dst, true);
        else t->point_msb(t->tables[idx], dst);
        dirty.push_back(idx);
      }
    }
    std::sort(dirty.begin(), dirty.end());
    dirty.erase(std::unique(dirty.begin(), dirty.end()), dirty.end());
    for (size_t idx : dirty)  // 144 bytes each, from pageable memory: staged by the runtime before the call returns
      SM_CUDA_TRY(cudaMemcpyAsync(t->tables_dev + idx, &t->tables[idx], sizeof(slicemoe_expert), cudaMemcpyHostToDevice, xs));
    SM_CUDA_TRY(cudaEventRecord(t->ev_copy, xs));
    SM_CUDA_TRY(cudaStreamWaitEvent(cs, t->ev_copy, 0));
  } catch (...) {
    return SLICEMOE_E_NOMEM;
  }
  return SLICEMOE_OK;
}

extern "C" int slicemoe_tier_sync(slicemoe_tier* t, void* compute_stream, void* copy_stream) {
  if (!t) return SLICEMOE_E_INVALID_ARG;
  cudaStream_t cs = (cudaStream_t)compute_stream, xs = (cudaStream_t)copy_stream;
  try {
    SM_CUDA_TRY(cudaEventRecord(t->ev_compute, cs));
    SM_CUDA_TRY(cudaStreamWaitEvent(xs, t->ev_compute, 0));
    // whatever the log holds is covered by the comparison below
    {
      int32_t el[64], ee[64];
      uint8_t il[64];
      while (slicemoe_dbsc_drain_evicted(t->cache, el, ee, il, 64) == 64) {
      }
    }
    t->transient.clear();
    std::vector<size_t> dirty;
    const int E = t->shape.n_experts;
    // first give back every slot whose slice the books no longer hold, then fetch what they hold and the pool lacks
    for (int pass = 0; pass < 2; ++pass) {
      for (int l = 0; l < t->n_layers; ++l) {
        for (int e = 0; e < E; ++e) {
          int has[2] = {0, 0};
          slicemoe_dbsc_contains(t->cache, l, e, &has[0], &has[1]);
          const uint64_t k = tier_key(l, e);
          const size_t idx = static_cast<size_t>(l) * E + e;
          for (int part = 0; part < 2; ++part) {
            auto& map = part ? t->lsb_slot : t->msb_slot;
            auto it = map.find(k);
            if (pass == 0 && it != map.end() && !has[part]) {
              t->free_slots.push_back(it->second);
              map.erase(it);
              if (part) t->point_lsb(t->tables[idx], t->pool, false);
              else t->point_msb(t->tables[idx], t->pool);
              dirty.push_back(idx);
            } else if (pass == 1 && it == map.end() && has[part]) {
              if (t->free_slots.empty()) return SLICEMOE_E_UNSUPPORTED;
              const int slot = t->free_slots.back();
              t->free_slots.pop_back();
              map[k] = slot;
              uint8_t* dst = t->pool + static_cast<size_t>(slot) * t->slot_bytes;
              const int rc = t->fetch(idx, part, dst, xs);
              if (rc != SLICEMOE_OK) return rc;
              if (part) t->point_lsb(t->tables[idx], dst, true);
              else t->point_msb(t->tables[idx], dst);
              dirty.push_back(idx);
            }
          }
        }
      }
    }
    std::sort(dirty.begin(), dirty.end());
    dirty.erase(std::unique(dirty.begin(), dirty.end()), dirty.end());
    for (size_t idx : dirty)
      SM_CUDA_TRY(cudaMemcpyAsync(t->tables_dev + idx, &t->tables[idx], sizeof(slicemoe_expert), cudaMemcpyHostToDevice, xs));
    SM_CUDA_TRY(cudaEventRecord(t->ev_copy, xs));
    SM_CUDA_TRY(cudaStreamWaitEvent(cs, t->ev_copy, 0));
  } catch (...) {
    return SLICEMOE_E_NOMEM;
  }
  return SLICEMOE_OK;
}

extern "C" int slicemoe_tier_stats(const slicemoe_tier* t, int64_t* bytes_copied, int64_t* copies, int64_t* free_slots) {
  if (!t) return SLICEMOE_E_INVALID_ARG;
  if (bytes_copied) *bytes_copied = t->bytes_copied;
  if (copies) *copies = t->copies;
  if (free_slots) *free_slots = static_cast<int64_t>(t->free_slots.size());
  return SLICEMOE_OK;
}
