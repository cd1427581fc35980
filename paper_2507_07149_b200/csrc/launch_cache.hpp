// What a launcher has to find out once per (kernel, device, dynamic shared-memory size): how many
// CTAs of a persistent kernel fit the device.  Plain C++ (no CUDA types), so that the host tests can
// exercise it with made-up device numbers; the query that fills an entry is passed in.
#pragma once
#include <map>
#include <mutex>
#include <tuple>

namespace daf {

class LaunchCache {
public:
    // Returns the remembered value for (kernel, device, dyn_smem); on the first request for a key
    // `query(&value)` computes it (an int error code other than 0 is passed through and nothing is
    // remembered).  Calls for different devices never share an entry.  Thread safe.
    template <typename Query> int get(const void *kernel, int device, int dyn_smem, int *value, Query query)
    {
        const Key key{kernel, device, dyn_smem};
        std::lock_guard<std::mutex> hold(mutex_);
        auto it = entries_.find(key);
        if (it == entries_.end()) {
            int v = 0;
            const int err = query(&v);
            if (err != 0) return err;
            it = entries_.emplace(key, v).first;
        }
        *value = it->second;
        return 0;
    }
    size_t size() const
    {
        std::lock_guard<std::mutex> hold(mutex_);
        return entries_.size();
    }

private:
    using Key = std::tuple<const void *, int, int>;
    mutable std::mutex mutex_;
    std::map<Key, int> entries_;
};

}  // namespace daf
