"""DRAM traffic of the dominant kernels as ncu counted it (dram__bytes_read.sum +
dram__bytes_write.sum per launch), kept in profiles/ncu_traffic.json together with a digest of the
kernel sources at the time of the capture.  bench.py reports an entry only while that digest still
matches: once a kernel source has changed, its counters are stale and the lookup returns None.

  python -m paper_2506_14435_b200.traffic add <workload> <stage> <tensor|stream> <bytes> <summary file>
  python -m paper_2506_14435_b200.traffic list
"""
from __future__ import annotations

import hashlib
import json
import os
import sys

_HERE = os.path.dirname(os.path.abspath(__file__))
_JSON = os.path.join(os.path.dirname(_HERE), "profiles", "ncu_traffic.json")

# the sources a stage's kernel is compiled from, per implementation
_SOURCES = {
    "tensor": ["umma_gemm.cu", "ptx_sm100.cuh", "mote_common.cuh"],
    "stream": ["decode_stream.cu", "mote_common.cuh"],
}


def source_digest(impl: str) -> str:
    h = hashlib.sha256()
    for name in _SOURCES[impl]:
        with open(os.path.join(_HERE, "csrc", name), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


def _load() -> list:
    if not os.path.exists(_JSON):
        return []
    with open(_JSON) as fh:
        return json.load(fh)["entries"]


def lookup(workload: str, stage: str, impl: str):
    """Bytes per launch for (workload, stage) on the implementation `impl`, or None when there is
    no capture or the kernel has changed since it was taken."""
    try:
        digest = source_digest(impl)
    except OSError:
        return None
    for e in _load():
        if e["workload"] == workload and e["stage"] == stage and e["impl"] == impl and e["digest"] == digest:
            return e["dram_bytes_per_launch"]
    return None


def add(workload: str, stage: str, impl: str, nbytes: float, summary: str) -> None:
    entries = [e for e in _load() if not (e["workload"] == workload and e["stage"] == stage and e["impl"] == impl)]
    entries.append({"workload": workload, "stage": stage, "impl": impl, "dram_bytes_per_launch": float(nbytes),
                    "summary": summary, "digest": source_digest(impl)})
    entries.sort(key=lambda e: (e["workload"], e["stage"], e["impl"]))
    with open(_JSON, "w") as fh:
        json.dump({"what": "ncu dram__bytes_read.sum + dram__bytes_write.sum per launch; digest = sha256 of the "
                           "kernel sources when captured (see paper_2506_14435_b200/traffic.py)",
                   "entries": entries}, fh, indent=1)
        fh.write("\n")


if __name__ == "__main__":
    if len(sys.argv) == 7 and sys.argv[1] == "add":
        add(sys.argv[2], sys.argv[3], sys.argv[4], float(sys.argv[5]), sys.argv[6])
    elif len(sys.argv) == 2 and sys.argv[1] == "list":
        for e in _load():
            ok = e["digest"] == source_digest(e["impl"])
            print(f'{e["workload"]:8s} {e["stage"]:16s} {e["impl"]:7s} {e["dram_bytes_per_launch"]:14.0f}  '
                  f'{"current" if ok else "STALE"}  {e["summary"]}')
    else:
        raise SystemExit(__doc__)
