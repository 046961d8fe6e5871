"""Small input builders shared by the test files (inputs only)."""
import numpy as np

PALETTE_1 = np.array([[0, 0, 0], [200, 100, 50]], np.uint8)
SKY = (127, 178, 229)


def cam_row(x, y, z, yaw, pitch, self_box=-1):
    row = np.zeros(6, np.int32)
    row[:5] = np.array([x, y, z, yaw, pitch], np.float32).view(np.int32)
    row[5] = self_box
    return row


def box_rows(items):
    """items: [((lo xyz), (hi xyz), material)] -> int32[n][8] in the C ABI's 32-byte box layout."""
    out = np.zeros((len(items), 8), np.int32)
    for n, (lo, hi, m) in enumerate(items):
        out[n, :6] = np.array(list(lo) + list(hi), np.float32).view(np.int32)
        out[n, 6] = m
    return out


def default_lut_intensities():
    """The default light (0.36, 0.80, 0.48) has unit length, so lit faces get 0.3 + 0.7*component."""
    return {"+x": 0.3 + 0.7 * 0.36, "+y": 0.3 + 0.7 * 0.80, "+z": 0.3 + 0.7 * 0.48,
            "-x": 0.3, "-y": 0.3, "-z": 0.3}
