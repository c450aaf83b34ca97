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


def kquants_blocks():
    """Parse kquants_handbuilt.txt -> {name: dict(fmt='q8_0'|'q6_k', bytes=uint8[...], w={index: value})}."""
    rules = {
        "(n-16)&255": lambda n: (n - 16) & 255, "128": lambda n: np.full_like(n, 128), "0": lambda n: np.zeros_like(n),
        "(n%16) | ((n//4)%16)<<4": lambda n: (n % 16) | (((n // 4) % 16) << 4), "(7*n+3)%256": lambda n: (7 * n + 3) % 256,
        "(n-8)&255": lambda n: (n - 8) & 255,
    }
    out, cur = {}, None
    for line in open(os.path.join(HERE, "kquants_handbuilt.txt")):
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
        fmt = name.split(".")[0]
        d = np.array([int(t, 16) for t in f["d_hex"].split()], np.uint8)
        if fmt == "q8_0":
            raw = np.concatenate([d, rules[f["payload_rule"]](np.arange(32)).astype(np.uint8)])
        else:
            raw = np.concatenate([rules[f["ql_rule"]](np.arange(128)).astype(np.uint8), rules[f["qh_rule"]](np.arange(64)).astype(np.uint8),
                                  rules[f["sc_rule"]](np.arange(16)).astype(np.uint8), d])
        blocks[name] = dict(fmt=fmt, bytes=raw, w={int(t.split(":")[0]): float(t.split(":")[1]) for t in f["w"].split()})
    return blocks
