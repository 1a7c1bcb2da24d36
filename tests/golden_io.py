"""Reader for the small text fixtures under tests/golden/ ('#' comments, a key line, then rows)."""
import os


def read_sections(path):
    sections, key = {}, None
    with open(path) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            if line[0].isalpha() and " " not in line and not line.startswith("a("):
                key = line
                sections[key] = []
            else:
                sections.setdefault(key, []).append(line.split())
    return sections


def golden(name):
    return os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", name)
