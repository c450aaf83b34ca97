"""Reader for the small text fixtures in this folder."""
import os

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))


def handbuilt_blocks():
    """Parse q4k_handbuilt.txt -> {name: dict(bytes=uint8[144], d, dmin, sc, m, w={index: value})}."""
    out, cur = {}, None
    for line in open(os.path.join(HERE, "q4k_handbuilt.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        if line.startswith("["):
            cur = line.strip("[]")
            out[cur] = {}
            continue
        key, val = line.split(":", 1)
        out[cur][key.strip()] = val.strip()
    blocks = {}
    for name, f in out.items():
        hdr = np.array([int(t, 16) for t in f["header_hex"].split()], np.uint8)
        n = np.arange(128)
        rule = f["qs_rule"]
        if rule == "255":
            qs = np.full(128, 255, np.uint8)
        elif rule == "n%16 | ((n//8)%16)<<4":
            qs = ((n % 16) | (((n // 8) % 16) << 4)).astype(np.uint8)
        else:
            raise ValueError(rule)
        blocks[name] = dict(
            bytes=np.concatenate([hdr, qs]),
            d=float(f["d"]), dmin=float(f["dmin"]),
            sc=[int(t) for t in f["sc"].split()], m=[int(t) for t in f["m"].split()],
            w={int(t.split(":")[0]): float(t.split(":")[1]) for t in f["w"].split()},
        )
    return blocks


def prp_schedules():
    """Parse prp_schedule.txt -> {name: dict(layers, window_sizes, rounds, w=[(round, device, first, last)], ...)}."""
    out, cur = {}, None
    for line in open(os.path.join(HERE, "prp_schedule.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        if line.startswith("["):
            cur = line.strip("[]")
            out[cur] = {"w": []}
            continue
        key, val = [t.strip() for t in line.split(":", 1)]
        nums = [int(t) for t in val.split()]
        if key == "w":
            out[cur]["w"].append(tuple(nums))
        else:
            out[cur][key] = nums if key == "window_sizes" else nums[0]
    return out
