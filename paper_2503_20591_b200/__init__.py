"""B200-native batched replica placement (after NotebookOS, arXiv 2503.20591).

`workloads` holds the seeded input generators; `binding` is the thin ctypes front
end of the CUDA library (libnbos.so, built in-tree by `build`). Importing this
package loads nothing heavy; the CUDA library is opened on first use and the call
fails loudly when it has not been built or no sm_100 device is present.
"""
