"""Regenerate ``rom_tables.json``: the frozen BOF4 / BOF5 / Split87 stand-in codebooks.

Run as ``python -m paper_2605_14929_b200.make_rom_tables``.  The tables are inputs to the sweep
(data, not method code); they are frozen so that every machine sees the same alphabet.
"""
import json

from . import inputs


def main() -> None:
    tables = inputs.build_rom_tables()
    with open(inputs.ROM_TABLE_PATH, "w") as f:
        json.dump(tables, f, indent=1)
    for k, v in tables.items():
        print(k, len(v), "ratio", round(inputs.lut_ratio(inputs.snap_bf16(v)), 2))


if __name__ == "__main__":
    main()
