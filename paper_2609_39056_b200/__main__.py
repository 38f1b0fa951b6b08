from . import build

if __name__ == "__main__":
    print(build.build(force=True))
