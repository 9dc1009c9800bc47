// Host-side helpers of the library (plain C++, no CUDA types): state that is set up once per device ordinal, and a
// small keyed cache with least-recently-used replacement.  Both are safe to call from several host threads.
#pragma once
#include <cstdint>
#include <cstring>
#include <mutex>

namespace hif8 {

constexpr int kMaxDevices = 64;

// One value of T per device ordinal, each initialised on first use by the caller's functor (run exactly once per
// device, with that device current).  Function attributes, SM counts and symbol addresses are per-device facts.
template <class T>
class PerDevice {
public:
    template <class Init>
    const T* get(int dev, Init&& init)
    {
        if (dev < 0 || dev >= kMaxDevices) return nullptr;
        std::call_once(once_[dev], [&] { init(dev, &val_[dev]); });
        return &val_[dev];
    }

private:
    std::once_flag once_[kMaxDevices];
    T val_[kMaxDevices];
};

// Cache of up to Cap values keyed by a trivially copyable Key (compared byte-wise; keys must be zero-initialised
// before their fields are set so that padding compares equal).  lookup_or_make copies the value out under the lock.
template <class Key, class Val, int Cap>
class LruCache {
public:
    // make(key, &val) -> bool builds the value of a key that is not cached; a failed build is not cached.
    template <class Make>
    bool lookup_or_make(const Key& key, Val* out, Make&& make)
    {
        std::lock_guard<std::mutex> lock(mu_);
        ++clock_;
        int victim = 0;
        for (int i = 0; i < Cap; i++) {
            if (used_[i] && std::memcmp(&keys_[i], &key, sizeof(Key)) == 0) {
                used_[i] = clock_;
                *out = vals_[i];
                ++hits_;
                return true;
            }
            if (used_[i] < used_[victim]) victim = i;
        }
        Val v;
        if (!make(key, &v)) return false;
        ++misses_;
        keys_[victim] = key;
        vals_[victim] = v;
        used_[victim] = clock_;
        *out = v;
        return true;
    }
    // value of a cached key, if any (counts as a use)
    bool find(const Key& key, Val* out)
    {
        std::lock_guard<std::mutex> lock(mu_);
        ++clock_;
        for (int i = 0; i < Cap; i++)
            if (used_[i] && std::memcmp(&keys_[i], &key, sizeof(Key)) == 0) {
                used_[i] = clock_;
                *out = vals_[i];
                return true;
            }
        return false;
    }
    // insert or overwrite
    void put(const Key& key, const Val& val)
    {
        std::lock_guard<std::mutex> lock(mu_);
        ++clock_;
        int victim = 0;
        for (int i = 0; i < Cap; i++) {
            if (used_[i] && std::memcmp(&keys_[i], &key, sizeof(Key)) == 0) { victim = i; break; }
            if (used_[i] < used_[victim]) victim = i;
        }
        keys_[victim] = key;
        vals_[victim] = val;
        used_[victim] = clock_;
    }
    uint64_t hits() const { return hits_; }
    uint64_t misses() const { return misses_; }

private:
    std::mutex mu_;
    Key keys_[Cap];
    Val vals_[Cap];
    uint64_t used_[Cap] = {};  // 0 = empty, else the clock value of the last use
    uint64_t clock_ = 0, hits_ = 0, misses_ = 0;
};

}  // namespace hif8
